// Verification with filtered target distributions (App. A.4 runs random sampling with top-k = 10 and
// top-p = 0.95): every distribution that Algorithm 1 tests against or samples from is softmax(z / T)
// restricted to its top_k largest logits (lowest token first on ties), then to the shortest prefix of
// those, in descending order, whose probability reaches top_p, and renormalised.
//
// Two launches of one kernel.  Phase 0 finds the top_k logits of the k+1 target rows; the last block
// of a sequence builds the filtered distributions, runs the acceptance loop (r <= Q'(c) / P_c), draws
// the extra token from row i* (Gumbel arg-max over the kept tokens, Philox noise keyed by the token as
// in verify.cu) and emits the tokens.  Phase 1 does the same for the k mask rows of group i* and
// writes the next candidates (their arg-maxes with P_c = 1, or samples from the filtered rows with
// their probabilities when candidates are sampled).
//
// SPACE_RESAMPLE_RESIDUAL_DRAFT keeps sampled candidates lossless (Sec. 3.2 claims an unchanged output
// distribution): phase 1 also writes every candidate's filtered distribution D as a list of top_k
// (token, probability) pairs, and phase 0 of the next step, after rejecting candidate i, draws the extra
// token from norm(max(0, Q - D_i)) -- one warp, its 32 lanes holding Q's kept tokens and D_i's entries.
//
// Top-k selection: every warp keeps a sorted list of at most 32 (logit, token) keys, one per lane, and
// a threshold (its last key); a logit above the threshold is inserted with one ballot and one shuffle.
// Keys are 64-bit words whose unsigned order is "larger logit, then lower token", so exact ties go to
// the lower token everywhere.  Warp lists meet in shared memory, block lists in a scratch array, and an
// arrival counter picks the block that finishes a sequence.
#include "common.cuh"
#include <math_constants.h>

namespace {

constexpr int FILT_THREADS = 256;
constexpr int FILT_MAX_CHUNKS = 16;
constexpr int FILT_MAX_K = 32;

struct FiltParams {
  int B, k, V, n_q, n_chunks, chunk, top_k, phase;
  int resample, eos_id;
  float top_p, c_t;                    // c_t = log2(e) / T
  uint32_t key0, key1;
  const void* logits; int64_t row_stride;
  const int32_t* cand; const float* cand_prob; const uint32_t* seq_id; const int32_t* kv_len;
  int32_t* n_accept; int32_t* out_tokens; int32_t* n_out; int32_t* next_cand; float* next_cand_prob;
  uint8_t* finished; int32_t* status;
  const int32_t* draft_tok; const float* draft_prob;      // [B, k, list_stride] or NULL (no lists)
  int32_t* next_draft_tok; float* next_draft_prob;        // [B, k, list_stride]
  int list_stride;
  unsigned long long* part;            // [B][k+1][FILT_MAX_CHUNKS][32]
  int* counter;                        // [B], self-resetting
};

__device__ __forceinline__ float fexp2(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }

__device__ __forceinline__ unsigned long long make_key(float v, int idx) {
  uint32_t u = __float_as_uint(v);
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  return ((unsigned long long)u << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)idx);
}
__device__ __forceinline__ void split_key(unsigned long long key, float& v, int& idx) {
  uint32_t u = (uint32_t)(key >> 32);
  u = (u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u;
  v = __uint_as_float(u);
  idx = (int)(0xFFFFFFFFu - (uint32_t)key);
}
__device__ __forceinline__ unsigned long long shfl64(unsigned long long x, int src) {
  const uint32_t lo = __shfl_sync(0xFFFFFFFFu, (uint32_t)x, src), hi = __shfl_sync(0xFFFFFFFFu, (uint32_t)(x >> 32), src);
  return ((unsigned long long)hi << 32) | lo;
}
// The warp's list: lane j < K holds the j-th largest key seen so far (0 = empty), lanes >= K hold 0.
// Inserts x (the same value in every lane) if it beats the K-th key.
__device__ __forceinline__ void list_insert(unsigned long long& mine, unsigned long long x, int K, int lane) {
  const int pos = __popc(__ballot_sync(0xFFFFFFFFu, mine > x));
  const uint32_t lo = __shfl_up_sync(0xFFFFFFFFu, (uint32_t)mine, 1), hi = __shfl_up_sync(0xFFFFFFFFu, (uint32_t)(mine >> 32), 1);
  if (pos < K) {
    if (lane == pos) mine = x;
    else if (lane > pos && lane < K) mine = ((unsigned long long)hi << 32) | lo;
  }
}

__device__ __forceinline__ float ld_logit(const float* p) { return *p; }
__device__ __forceinline__ float ld_logit(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// 16 bytes of logits as floats
__device__ __forceinline__ void unpack16(const uint4& v, float (&f)[4], const float*) {
  f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
}
__device__ __forceinline__ void unpack16(const uint4& v, float (&f)[8], const __nv_bfloat16*) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) { f[2 * i] = __uint_as_float(w[i] << 16); f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u); }
}

// VECTOR: the row and the chunk start are 16-byte aligned (the launcher checks): every lane fetches four
// 16-byte pieces per sweep, all in flight together, instead of one logit at a time.
template <typename T, bool VECTOR>
__global__ void __launch_bounds__(FILT_THREADS) verify_filter_kernel(const FiltParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.z, r = blockIdx.y, ch = blockIdx.x;
  const int k1 = p.k + 1, K = p.top_k;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_rows = p.phase == 0 ? k1 : p.k;
  const int i_star0 = p.phase == 0 ? 0 : max(0, min(p.n_accept[b], p.k));
  const int brow = p.phase == 0 ? r * k1 : i_star0 * k1 + r + 1;          // target row r, or mask row (i*, r+1)
  const T* row = reinterpret_cast<const T*>(p.logits) + ((int64_t)b * p.n_q + brow) * p.row_stride;
  const int begin = ch * p.chunk, end = min(p.V, begin + p.chunk);

  // ---- this warp's top-K of its share of the chunk ------------------------------------
  unsigned long long mine = 0ull;
  int scalar_from = begin;                                  // what the one-by-one loop below still has to look at
  if (VECTOR) {
    constexpr int N = 16 / (int)sizeof(T), U = 4;
    const int full_end = begin + ((end - begin) / N) * N;
    constexpr int stride = FILT_THREADS * N;
    unsigned long long tau = 0ull;                          // the warp's K-th key so far (0: fewer than K keys)
    for (int xw = begin + warp * 32 * N; xw < full_end; xw += U * stride) {   // (the same trip count in every lane)
      uint4 v[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int x = xw + lane * N + u * stride;
        v[u] = x < full_end ? __ldg(reinterpret_cast<const uint4*>(row + x)) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int x = xw + lane * N + u * stride;
        float f[N];
        unpack16(v[u], f, (const T*)nullptr);
#pragma unroll
        for (int i = 0; i < N; ++i) {
          const unsigned long long key = x < full_end ? make_key(f[i], x + i) : 0ull;
          unsigned pass = __ballot_sync(0xFFFFFFFFu, key > tau);
          while (pass) {
            const int src = __ffs(pass) - 1;
            pass &= pass - 1;
            list_insert(mine, shfl64(key, src), K, lane);
            tau = shfl64(mine, K - 1);
          }
        }
      }
    }
    scalar_from = full_end;                                 // (fewer than N logits, looked at by every warp: keys are unique, a
  }                                                         //  second look at one changes nothing -- but only warp 0 does it)
  for (int x0 = scalar_from + (VECTOR ? 0 : warp * 32); x0 < end && (!VECTOR || warp == 0); x0 += VECTOR ? 32 : FILT_THREADS) {
    const int x = x0 + lane;
    const unsigned long long key = x < end ? make_key(ld_logit(row + x), x) : 0ull;
    const unsigned long long tau = shfl64(mine, K - 1);
    unsigned pass = __ballot_sync(0xFFFFFFFFu, key > tau);
    while (pass) {
      const int src = __ffs(pass) - 1;
      pass &= pass - 1;
      list_insert(mine, shfl64(key, src), K, lane);
    }
  }
  // ---- block list: warp 0 merges the eight warp lists ----------------------------------
  __shared__ unsigned long long sh_list[FILT_THREADS / 32][32];
  sh_list[warp][lane] = mine;
  __syncthreads();
  unsigned long long* part = p.part + (((int64_t)b * k1 + r) * FILT_MAX_CHUNKS) * 32;
  if (warp == 0) {
    for (int w = 1; w < FILT_THREADS / 32; ++w) {
      const unsigned long long other = sh_list[w][lane];
      for (int j = 0; j < K; ++j) {
        const unsigned long long x = shfl64(other, j);
        if (x == 0ull) break;                               // (uniform: x is the same in every lane)
        list_insert(mine, x, K, lane);
      }
    }
    *reinterpret_cast<volatile unsigned long long*>(part + ch * 32 + lane) = mine;
  }
  // ---- arrival: the last block of the sequence finishes it -------------------------------
  __shared__ int sh_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const int prev = atomicAdd(p.counter + b, 1);
    sh_last = prev == n_rows * p.n_chunks - 1;
    if (sh_last) p.counter[b] = 0;
  }
  __syncthreads();
  if (!sh_last) return;
  __threadfence();

  // ---- last block: warp w builds the filtered distribution of row w ----------------------
  __shared__ int sh_ok[SPACE_MAX_K + 1];
  __shared__ int sh_bits;
  if (threadIdx.x == 0) sh_bits = 0;
  const bool with_lists = p.resample == SPACE_RESAMPLE_RESIDUAL_DRAFT;
  const bool literal = p.resample == SPACE_RESAMPLE_PAPER_LITERAL || with_lists;   // candidates are sampled
  const uint32_t seq = p.seq_id ? p.seq_id[b] : (uint32_t)b;
  const int L = p.kv_len ? p.kv_len[b] : 0;
  float z = 0.f, q = 0.f; int idx = -1; bool keep = false;
  if (warp < n_rows) {
    unsigned long long lst = 0ull;
    const unsigned long long* pr = p.part + (((int64_t)b * k1 + warp) * FILT_MAX_CHUNKS) * 32;
    for (int c = 0; c < p.n_chunks; ++c) {
      const unsigned long long other = __ldcg(pr + c * 32 + lane);
      for (int j = 0; j < K; ++j) {
        const unsigned long long x = shfl64(other, j);
        if (x == 0ull) break;
        list_insert(lst, x, K, lane);
      }
    }
    const bool valid = lst != 0ull;
    if (valid) split_key(lst, z, idx);
    // temperature, then softmax over the top-k, then the shortest prefix that reaches top_p
    const float s = z * p.c_t;
    const float s0 = __shfl_sync(0xFFFFFFFFu, s, 0);
    float pj = valid ? fexp2(s - s0) : 0.f;
    float tot = pj;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xFFFFFFFFu, tot, o);
    pj /= tot;
    float cum = pj;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const float up = __shfl_up_sync(0xFFFFFFFFu, cum, o);
      if (lane >= o) cum += up;
    }
    float before = __shfl_up_sync(0xFFFFFFFFu, cum, 1);     // probability of the tokens before this one
    if (lane == 0) before = 0.f;
    keep = valid && (lane == 0 || p.top_p >= 1.f || before < p.top_p);   // top_p = 1: no nucleus cut
    float ksum = keep ? pj : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ksum += __shfl_xor_sync(0xFFFFFFFFu, ksum, o);
    q = keep ? pj / ksum : 0.f;
  }
  __syncthreads();                                          // sh_bits is zero for everyone

  if (p.phase == 0) {
    // acceptance test of candidate c_{t+1} against the filtered law of target row t (warp t)
    if (warp < p.k) {
      const int c = p.cand[b * p.k + warp];
      const bool in_range = c >= 0 && c < p.V;
      const unsigned hit = __ballot_sync(0xFFFFFFFFu, keep && idx == c);
      const float qc = hit ? __shfl_sync(0xFFFFFFFFu, q, __ffs(hit) - 1) : 0.f;
      if (lane == 0) {
        if (!in_range) atomicOr(&sh_bits, SPACE_ST_BAD_CANDIDATE);
        const Philox4 w = philox4x32_10(0u, PURPOSE_ACCEPT, seq, (uint32_t)(L + warp + 1), p.key0, p.key1);
        const float pc = p.cand_prob[b * p.k + warp];
        sh_ok[warp] = in_range && pc > 0.f && uniform_open(w.x) * pc <= qc;   // r <= Q'/P_c  <=>  r P_c <= Q'
      }
    }
    __syncthreads();
    int i_star = 0;
    while (i_star < p.k && sh_ok[i_star]) ++i_star;
    if (warp == i_star) {
      // extra token: Gumbel arg-max over the kept tokens of row i*, the rejected point-mass candidate left out
      int exclude = -1;
      if (!literal && i_star < p.k && p.cand_prob[b * p.k + i_star] == 1.0f) exclude = p.cand[b * p.k + i_star];
      float sc = -CUDART_INF_F;
      // compact draft distribution of the rejected candidate: the weight of a kept token is
      // max(0, Q - D); Q itself when nothing was rejected, there are no lists, or nothing is left
      float wq = q;
      bool residual = false;
      if (with_lists && i_star < p.k && p.draft_tok) {
        int dt = -1; float dp = 0.f;
        if (lane < p.list_stride) {
          dt = p.draft_tok[((int64_t)b * p.k + i_star) * p.list_stride + lane];
          dp = p.draft_prob[((int64_t)b * p.k + i_star) * p.list_stride + lane];
          if (dt < 0 || dt >= p.V || !(dp > 0.f) || !(dp < CUDART_INF_F)) { dt = -1; dp = 0.f; }
        }
        float d = 0.f;
        for (int j = 0; j < p.list_stride; ++j) {
          const int tj = __shfl_sync(0xFFFFFFFFu, dt, j);
          const float pj2 = __shfl_sync(0xFFFFFFFFu, dp, j);
          if (tj == idx) d += pj2;
        }
        const float res = keep ? fmaxf(q - d, 0.f) : 0.f;
        residual = __any_sync(0xFFFFFFFFu, res > 0.f);
        if (residual) wq = res;
      }
      if (keep && idx != exclude && (!residual || wq > 0.f)) {
        const Philox4 ph = philox4x32_10((uint32_t)(idx >> 2), PURPOSE_TOKEN, seq, (uint32_t)(L + i_star + 1), p.key0, p.key1);
        const uint32_t w4[4] = {ph.x, ph.y, ph.z, ph.w};
        const float g = gumbel2_from_uniform(uniform_open(w4[idx & 3]));
        sc = with_lists ? fast_log2(wq) + g : fmaf(z, p.c_t, g);
      }
      int bi = keep ? idx : 0x7FFFFFFF;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float os = __shfl_xor_sync(0xFFFFFFFFu, sc, o);
        const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, o);
        if (os > sc || (os == sc && oi < bi)) { sc = os; bi = oi; }
      }
      const int bonus = bi;
      const int j = lane;
      const int tok = (j < i_star) ? p.cand[b * p.k + min(j, p.k - 1)] : (j == i_star ? bonus : -1);
      const bool is_eos = p.eos_id >= 0 && j <= i_star && tok == p.eos_id;
      const unsigned eos_mask = __ballot_sync(0xFFFFFFFFu, is_eos && j < k1);
      const int n_out = eos_mask ? __ffs(eos_mask) - 1 : i_star + 1;
      if (j < k1) p.out_tokens[b * k1 + j] = (j < n_out) ? tok : -1;
      if (j == 0) {
        p.n_accept[b] = i_star;
        p.n_out[b] = n_out;
        p.finished[b] = (uint8_t)(eos_mask != 0);
        if (p.status && sh_bits) atomicOr(p.status + b, sh_bits);
      }
    }
  } else if (warp < p.k) {
    // next candidate o = warp + 1 from mask row (i*, o)
    int tok; float pr;
    if (!literal) {                                         // point-mass draft: the row's arg-max, P_c = 1
      tok = __shfl_sync(0xFFFFFFFFu, idx, 0); pr = 1.f;
    } else {
      float sc = -CUDART_INF_F;
      if (keep) {
        const Philox4 ph = philox4x32_10((uint32_t)(idx >> 2), PURPOSE_DRAFT, seq, (uint32_t)(L + i_star0 + 1 + warp + 1),
                                         p.key0, p.key1);
        const uint32_t w4[4] = {ph.x, ph.y, ph.z, ph.w};
        sc = fmaf(z, p.c_t, gumbel2_from_uniform(uniform_open(w4[idx & 3])));
      }
      int bi = keep ? idx : 0x7FFFFFFF; float bq = q;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float os = __shfl_xor_sync(0xFFFFFFFFu, sc, o);
        const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, o);
        const float oq = __shfl_xor_sync(0xFFFFFFFFu, bq, o);
        if (os > sc || (os == sc && oi < bi)) { sc = os; bi = oi; bq = oq; }
      }
      tok = bi; pr = bq;
    }
    if (lane == 0) { p.next_cand[b * p.k + warp] = tok; p.next_cand_prob[b * p.k + warp] = pr; }
    if (with_lists && lane < p.list_stride) {               // the row's filtered distribution, descending
      p.next_draft_tok[((int64_t)b * p.k + warp) * p.list_stride + lane] = keep ? idx : -1;
      p.next_draft_prob[((int64_t)b * p.k + warp) * p.list_stride + lane] = keep ? q : 0.f;
    }
  }
}

}  // namespace

size_t verify_filter_scratch_bytes(int max_batch, int k_max) {
  return (size_t)max_batch * (k_max + 1) * FILT_MAX_CHUNKS * 32 * sizeof(unsigned long long);
}

int launch_verify_filtered(space_ctx* ctx, const space_verify_args* a, cudaStream_t st) {
  if (a->top_k < 1 || a->top_k > FILT_MAX_K || !(a->top_p > 0.f) || a->top_p > 1.f) return SPACE_E_INVALID_ARG;
  FiltParams p;
  memset(&p, 0, sizeof(p));
  p.B = a->batch; p.k = a->k; p.V = a->vocab; p.n_q = (a->k + 1) * (a->k + 1);
  p.top_k = a->top_k < a->vocab ? a->top_k : a->vocab; p.top_p = a->top_p;
  p.resample = a->resample; p.eos_id = a->eos_id;
  p.c_t = 1.4426950408889634f / a->temperature;
  p.key0 = (uint32_t)(a->seed & 0xFFFFFFFFull); p.key1 = (uint32_t)(a->seed >> 32);
  p.logits = a->logits; p.row_stride = a->logits_row_stride;
  p.cand = a->cand; p.cand_prob = a->cand_prob; p.seq_id = a->seq_id; p.kv_len = a->kv_len;
  p.n_accept = a->n_accept; p.out_tokens = a->out_tokens; p.n_out = a->n_out; p.next_cand = a->next_cand;
  p.next_cand_prob = a->next_cand_prob; p.finished = a->finished; p.status = a->status;
  p.draft_tok = a->draft_tok; p.draft_prob = a->draft_prob;
  p.next_draft_tok = a->next_draft_tok; p.next_draft_prob = a->next_draft_prob; p.list_stride = a->top_k;
  p.part = reinterpret_cast<unsigned long long*>(ctx->vtopk);
  // about two blocks per SM over the (k+1) rows of every sequence, at least 8192 logits per block
  const int rows = a->batch * (a->k + 1);
  int nc = (2 * ctx->sm_count + rows - 1) / rows;   // (4, 8, 16 per SM measured slower: every block starts from an empty list)
  const int max_nc = (a->vocab + 8191) / 8192;
  if (nc > max_nc) nc = max_nc;
  if (nc > FILT_MAX_CHUNKS) nc = FILT_MAX_CHUNKS;
  if (nc < 1) nc = 1;
  p.chunk = (((a->vocab + nc - 1) / nc + 7) / 8) * 8;       // chunk starts stay 16-byte aligned
  p.n_chunks = (a->vocab + p.chunk - 1) / p.chunk;
  const int esz = a->logits_dtype == SPACE_DTYPE_F32 ? 4 : 2;
  const bool vector = ((uintptr_t)a->logits % 16 == 0) && ((a->logits_row_stride * esz) % 16 == 0);
  for (int phase = 0; phase < 2; ++phase) {
    p.phase = phase;
    p.counter = ctx->counters + (phase == 0 ? 0 : ctx->cfg.max_batch);
    const dim3 grid(p.n_chunks, phase == 0 ? a->k + 1 : a->k, a->batch);
    ProfScope ps(ctx, phase == 0 ? SPACE_K_VERIFY_TARGET : SPACE_K_VERIFY_EMIT, st);
    if (a->logits_dtype == SPACE_DTYPE_F32) {
      if (vector) launch_pdl(verify_filter_kernel<float, true>, grid, dim3(FILT_THREADS), 0, st, p);
      else launch_pdl(verify_filter_kernel<float, false>, grid, dim3(FILT_THREADS), 0, st, p);
    } else {
      if (vector) launch_pdl(verify_filter_kernel<__nv_bfloat16, true>, grid, dim3(FILT_THREADS), 0, st, p);
      else launch_pdl(verify_filter_kernel<__nv_bfloat16, false>, grid, dim3(FILT_THREADS), 0, st, p);
    }
  }
  ctx->launches += 2;
  return cuda_ok(cudaGetLastError());
}
