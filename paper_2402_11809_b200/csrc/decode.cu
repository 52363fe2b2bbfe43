// Device-resident state of the decoding loop of Algorithm 1.
//
// Algorithm 1 keeps O (the tokens so far), L_c and P_c (the candidates and their probabilities)
// from one model call to the next, builds the extended input of the next call (Eq. 4) with its
// position ids (Sec. 3.2) and returns at the first <EOS>.  The two kernels here keep that state
// on the GPU, so that the caller's model, space_attn_step, space_verify_commit and the state
// update can follow one another on a stream (or in one CUDA graph) without a host round trip:
//   decode_begin_kernel    O = {}, L_c = [0]*k, P_c = [+inf]*k, block rows of the first step
//   decode_advance_kernel  append the step's tokens, latch <EOS>, carry the new candidates and
//                          the new length, write the block rows of the next step
// One thread block per sequence; a handful of integers each.
#include "common.cuh"
#include <math_constants.h>

namespace {

struct DecodeParams {
  space_decode_state s;
  int n_q;
  signed char relpos[SPACE_MAX_ROWS];  // position id of block row i minus the verified length (Sec. 3.2)
  const int32_t* first_token;          // begin: last token of the prompt
  const int32_t* out_tokens; const int32_t* n_out; const int32_t* next_cand; const float* next_cand_prob;
  const uint8_t* step_finished; const int32_t* kv_len_next;
};

// Block rows of the next model call: row g(k+1)+o is the last verified token (g = 0, o = 0), the
// candidate c_g (o = 0) or the mask token (o >= 1); positions follow the visibility rule.
__device__ __forceinline__ void write_block_rows(const DecodeParams& p, int b, int last_token, int L) {
  const int k1 = p.s.k + 1;
  for (int i = threadIdx.x; i < p.n_q; i += blockDim.x) {
    const int g = i / k1, o = i - g * k1;
    int tok = p.s.mask_token_id;
    if (o == 0) tok = (g == 0) ? last_token : p.s.cand[b * p.s.k + g - 1];
    p.s.block_tokens[b * p.n_q + i] = tok;
    p.s.block_pos[b * p.n_q + i] = L + p.relpos[i];
  }
}

__global__ void __launch_bounds__(64) decode_begin_kernel(const DecodeParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  if (threadIdx.x < p.s.k) {                                // Algorithm 1: L_c = [0]*k, P_c = [+inf]*k
    p.s.cand[b * p.s.k + threadIdx.x] = 0;
    p.s.cand_prob[b * p.s.k + threadIdx.x] = CUDART_INF_F;
  }
  const int last = p.first_token[b];
  if (threadIdx.x == 0) {
    p.s.n_tokens[b] = 0;
    p.s.finished[b] = 0;
    p.s.last_token[b] = last;
  }
  __syncthreads();                                          // the candidates are read back below
  write_block_rows(p, b, last, p.s.kv_len[b]);
}

__global__ void __launch_bounds__(64) decode_advance_kernel(const DecodeParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  if (p.s.finished[b]) return;                              // latched: the step's results are dropped
  const int k = p.s.k;
  const int have = p.s.n_tokens[b];
  int n = p.n_out[b];
  n = max(0, min(n, k + 1));
  const int room = p.s.max_tokens - have;
  const bool full = n >= room;                              // the output buffer ends the sequence too
  const int n_take = min(n, room);
  if (threadIdx.x < n_take) p.s.tokens[(int64_t)b * p.s.max_tokens + have + threadIdx.x] = p.out_tokens[b * (k + 1) + threadIdx.x];
  const bool done = p.step_finished[b] != 0 || full;
  const int last = n > 0 ? p.out_tokens[b * (k + 1) + n - 1] : p.s.last_token[b];
  const int L = p.kv_len_next[b];
  if (!done && threadIdx.x < k) {                           // the candidates of the next step
    p.s.cand[b * k + threadIdx.x] = p.next_cand[b * k + threadIdx.x];
    p.s.cand_prob[b * k + threadIdx.x] = p.next_cand_prob[b * k + threadIdx.x];
  }
  __syncthreads();                                          // every thread has read the old state
  if (threadIdx.x == 0) {
    p.s.n_tokens[b] = have + n_take;
    if (done) p.s.finished[b] = 1;
    else { p.s.last_token[b] = last; p.s.kv_len[b] = L; }
  }
  if (!done) write_block_rows(p, b, last, L);
}

int fill(space_ctx* ctx, const space_decode_state* s, DecodeParams* p) {
  if (s->batch < 0 || s->batch > ctx->cfg.max_batch) return SPACE_E_WORKSPACE;
  if (s->k < 1 || s->k > ctx->cfg.k_max) return SPACE_E_INVALID_ARG;
  if (s->max_tokens < 1) return SPACE_E_INVALID_ARG;
  if (s->mask_variant != SPACE_MASK_SAME_GROUP && s->mask_variant != SPACE_MASK_EQ5_LITERAL) return SPACE_E_INVALID_ARG;
  if (s->batch == 0) return SPACE_OK;
  if (!s->tokens || !s->n_tokens || !s->last_token || !s->cand || !s->cand_prob || !s->kv_len || !s->finished ||
      !s->block_tokens || !s->block_pos)
    return SPACE_E_INVALID_ARG;
  memset(p, 0, sizeof(*p));
  p->s = *s;
  space_layout_t lay;
  const int rc = space_layout(s->k, s->mask_variant, &lay);
  if (rc != SPACE_OK) return rc;
  p->n_q = lay.n_q;
  for (int i = 0; i < lay.n_q; ++i) p->relpos[i] = (signed char)lay.relpos[i];
  return SPACE_OK;
}

}  // namespace

extern "C" {

int space_decode_begin(space_ctx* ctx, const space_decode_state* state, const int32_t* last_prompt_token, void* stream) {
  if (!ctx || !state) return SPACE_E_INVALID_ARG;
  DecodeParams p;
  const int rc = fill(ctx, state, &p);
  if (rc != SPACE_OK || state->batch == 0) return rc;
  if (!last_prompt_token) return SPACE_E_INVALID_ARG;
  if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return SPACE_E_CUDA;
  p.first_token = last_prompt_token;
  launch_pdl(decode_begin_kernel, dim3(state->batch), dim3(64), 0, (cudaStream_t)stream, p);
  ctx->launches += 1;
  return cuda_ok(cudaGetLastError());
}

int space_decode_advance(space_ctx* ctx, const space_decode_state* state, const int32_t* out_tokens,
                         const int32_t* n_out, const int32_t* next_cand, const float* next_cand_prob,
                         const uint8_t* step_finished, const int32_t* kv_len_next, void* stream) {
  if (!ctx || !state) return SPACE_E_INVALID_ARG;
  DecodeParams p;
  const int rc = fill(ctx, state, &p);
  if (rc != SPACE_OK || state->batch == 0) return rc;
  if (!out_tokens || !n_out || !next_cand || !next_cand_prob || !step_finished || !kv_len_next) return SPACE_E_INVALID_ARG;
  if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return SPACE_E_CUDA;
  p.out_tokens = out_tokens; p.n_out = n_out; p.next_cand = next_cand; p.next_cand_prob = next_cand_prob;
  p.step_finished = step_finished; p.kv_len_next = kv_len_next;
  launch_pdl(decode_advance_kernel, dim3(state->batch), dim3(64), 0, (cudaStream_t)stream, p);
  ctx->launches += 1;
  return cuda_ok(cudaGetLastError());
}

}  // extern "C"
