// Verification and emission kernels (Algorithm 1 after the model call, Sec. 3.2).
//
// Two launches per step.
//   verify_target_kernel  streams the k+1 target rows (real token of every
//       sub-block) once: per row the maximum, the lowest-index arg-max and the
//       sum of exp((z - max)/T).  The last block to finish a sequence runs the
//       acceptance loop of Algorithm 1 and stores i*.
//   verify_emit_kernel    streams the k mask rows of group i* (the next
//       candidates) and, in sampling mode, the target row i* once more for the
//       extra token a (Gumbel arg-max with Philox noise).  The last block of a
//       sequence assembles the emitted tokens, the <EOS> cut and the new
//       candidates with their probabilities.
// Each row is cut into chunks so that small batches still fill the GPU; chunk
// results meet in a small scratch array and an arrival counter (reset by the
// last block) decides who finishes the sequence.
//
// Small greedy problems (all (k+1)^2 rows of the batch within 64 MB; measured: at
// 37 MB one launch still beats two by 6 us) are
// latency bound, not bandwidth bound: for them verify_fused_kernel streams
// every row in one launch and the last block of a sequence picks i* and the
// mask rows of group i* from the per-row results, which removes the second
// launch and its dependent round trips at the price of reading rows that the
// two-launch path skips.
#include "common.cuh"
#include <math_constants.h>

namespace {

constexpr int64_t SPACE_FUSED_MAX_BYTES = 64ll << 20;

struct VerifyParams {
  int B, k, V, n_q, n_chunks, chunk;
  int n_chunks_g, chunk_g;   // the row with Gumbel noise is cut finer (several times the work per logit)
  int mode, resample, eos_id;
  float c_t;                 // log2(e) / T   (target rows, sampled rows)
  float inv_t;               // 1 / T
  uint32_t key0, key1;
  const void* logits;
  int64_t row_stride;
  const int32_t* cand;
  const float* cand_prob;
  const uint32_t* seq_id;
  const int32_t* kv_len;
  int32_t* n_accept;
  int32_t* out_tokens;
  int32_t* n_out;
  int32_t* next_cand;
  float* next_cand_prob;
  uint8_t* finished;
  int32_t* status;
  VerifyPartial* part;       // [B][k+2][n_chunks]
  VerifyRow* rows;           // [B][k+1]
  int* counter_a;            // [B]
  int* counter_b;            // [B]
  int do_commit;             // the kernels also move the accepted cache rows (space_verify_commit)
  CommitParams cm;
};

// 2^x by the hardware approximation (relative error about 2^-22: far inside the
// 1e-4 bands the sums and probabilities are compared with)
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

struct Stat {                // running statistics of a set of logits
  float m, s;  int idx;      // max, sum exp2((z-m)*c), arg-max (lowest index)
  float gs;    int gidx;     // best Gumbel-perturbed score and its index
};

__device__ __forceinline__ Stat stat_empty() {
  return Stat{-CUDART_INF_F, 0.f, 0x7FFFFFFF, -CUDART_INF_F, 0x7FFFFFFF};
}

__device__ __forceinline__ void stat_merge(Stat& a, const Stat& b, float c) {
  if (b.m > a.m || (b.m == a.m && b.idx < a.idx)) a.idx = b.idx;
  const float m = fmaxf(a.m, b.m);
  if (m > -CUDART_INF_F) {
    const float sa = (a.m > -CUDART_INF_F) ? a.s * fast_exp2((a.m - m) * c) : 0.f;
    const float sb = (b.m > -CUDART_INF_F) ? b.s * fast_exp2((b.m - m) * c) : 0.f;
    a.s = sa + sb;
  }
  a.m = m;
  if (b.gs > a.gs || (b.gs == a.gs && b.gidx < a.gidx)) { a.gs = b.gs; a.gidx = b.gidx; }
}

__device__ __forceinline__ float load_logit(const float* p) { return *p; }
__device__ __forceinline__ float load_logit(const __nv_bfloat16* p) { return __bfloat162float(*p); }

template <typename T> struct Vec;
template <> struct Vec<float> {
  static constexpr int N = 4;
  static constexpr uint32_t NEG_INF = 0xFF800000u;          // raw word that converts to -inf
  static __device__ __forceinline__ void convert(const uint4& x, float* v) {
    v[0] = __uint_as_float(x.x); v[1] = __uint_as_float(x.y);
    v[2] = __uint_as_float(x.z); v[3] = __uint_as_float(x.w);
  }
};
template <> struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  static constexpr uint32_t NEG_INF = 0xFF80FF80u;
  static __device__ __forceinline__ void convert(const uint4& x, float* v) {
    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i]     = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
};

// One logit (the ragged ends of a chunk and unaligned rows).
// What a scan keeps of its logits: nothing (the noisy arg-max alone), the maximum with its
// lowest-index arg-max, or those and the sum of exp((z - max) c).
enum { STAT_NONE = 0, STAT_MAX = 1, STAT_SUM = 2 };

template <bool GUMBEL, int STATS>
__device__ __forceinline__ void fold_one(Stat& st, float v, int x, float c, int exclude,
                                         uint32_t key0, uint32_t key1, uint32_t purpose,
                                         uint32_t seq, uint32_t pos) {
  if (STATS == STAT_SUM) {
    if (v > st.m) {
      st.s = (st.m > -CUDART_INF_F) ? st.s * fast_exp2((st.m - v) * c) : 0.f;
      st.idx = x;
      st.m = v;
    }
    if (st.m > -CUDART_INF_F) st.s += fast_exp2(fmaf(v, c, -st.m * c));
  } else if (STATS == STAT_MAX) {
    if (v > st.m) { st.idx = x; st.m = v; }
  }
  if (GUMBEL) {
    // noise of token x: lane x&3 of the Philox block with counter word x>>2
    const Philox4 r = philox4x32_10((uint32_t)(x >> 2), purpose, seq, pos, key0, key1);
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
    const float sc = (x == exclude) ? -CUDART_INF_F : fmaf(v, c, gumbel2_from_uniform(uniform_open(w[x & 3])));
    if (sc > st.gs) { st.gs = sc; st.gidx = x; }
  }
}

// (max, lowest arg-max, sum of exp2((z - max) c)) of U vectors of N logits, the
// first at index x0, the u-th `stride` further: one maximum and one rescale per
// call, then independent exponentials and tree sums.  -inf entries (slots past the
// end of the chunk) change neither the maximum nor the sum.  st.idx is left at the first
// index of the vector that holds the maximum (see scan_chunk).
template <int U, int N, bool SUMS>
__device__ __forceinline__ void fold_stats(Stat& st, const float (&v)[U][N], int x0, int stride, float c) {
  float vm[U];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    float a[N];
#pragma unroll
    for (int i = 0; i < N; ++i) a[i] = v[u][i];
#pragma unroll
    for (int w = N / 2; w > 0; w >>= 1)
#pragma unroll
      for (int i = 0; i < w; ++i) a[i] = fmaxf(a[i], a[i + w]);
    vm[u] = a[0];
  }
  float vmax = vm[0];
#pragma unroll
  for (int u = 1; u < U; ++u) vmax = fmaxf(vmax, vm[u]);
  if (vmax > st.m) {
    if (SUMS) st.s = (st.m > -CUDART_INF_F) ? st.s * fast_exp2((st.m - vmax) * c) : 0.f;
    // first vector that holds the new maximum (walk backwards, the last hit wins); which of
    // its N logits it is gets settled once, at the end of the chunk (this branch is taken in
    // almost every sweep of a short chunk, so it stays small)
#pragma unroll
    for (int u = U - 1; u >= 0; --u)
      if (vm[u] == vmax) st.idx = x0 + u * stride;
    st.m = vmax;
  }
  if (SUMS && st.m > -CUDART_INF_F) {
    const float nmc = -st.m * c;                            // exp2(z*c - m*c): exponent error below 1e-5
    float su[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float e[N];
#pragma unroll
      for (int i = 0; i < N; ++i) e[i] = fast_exp2(fmaf(v[u][i], c, nmc));
#pragma unroll
      for (int w = N / 2; w > 0; w >>= 1)
#pragma unroll
        for (int i = 0; i < w; ++i) e[i] += e[i + w];
      su[u] = e[0];
    }
    float tot = su[0];
#pragma unroll
    for (int u = 1; u < U; ++u) tot += su[u];
    st.s += tot;
  }
}

// Best Gumbel-perturbed score of N logits starting at index x0 (a multiple of 4).
// A -inf logit (also the excluded token, set to -inf by the caller) never wins.
template <int N>
__device__ __forceinline__ void fold_gumbel(Stat& st, const float* v, int x0, float c,
                                            uint32_t key0, uint32_t key1, uint32_t purpose,
                                            uint32_t seq, uint32_t pos) {
#pragma unroll
  for (int i0 = 0; i0 < N; i0 += 4) {
    const Philox4 r = philox4x32_10((uint32_t)((x0 + i0) >> 2), purpose, seq, pos, key0, key1);
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
    float sc[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) sc[j] = fmaf(v[i0 + j], c, gumbel2_from_uniform(uniform_open(w[j])));
    // best of the four (lowest index on ties), then one update of the running best
    float b01 = sc[0]; int i01 = 0;
    if (sc[1] > b01) { b01 = sc[1]; i01 = 1; }
    float b23 = sc[2]; int i23 = 2;
    if (sc[3] > b23) { b23 = sc[3]; i23 = 3; }
    if (b23 > b01) { b01 = b23; i01 = i23; }
    if (b01 > st.gs) { st.gs = b01; st.gidx = x0 + i0 + i01; }
  }
}

// Statistics of logits [begin, end) of one row.  STATS: maximum, arg-max and sum;
// GUMBEL: the best noisy score (token `exclude` left out).  With VECTOR, `begin`
// is a multiple of the vector length and the row is 16-byte aligned.
template <typename T, bool VECTOR, bool GUMBEL, int STATS>
__device__ Stat scan_chunk(const T* row, int begin, int end, float c, int exclude,
                           uint32_t key0, uint32_t key1, uint32_t purpose, uint32_t seq,
                           uint32_t pos) {
  Stat st = stat_empty();
  if (VECTOR) {
    constexpr int N = Vec<T>::N;
    constexpr int U = 4;                                    // independent 16-byte loads in flight per thread
    // the tail shorter than N is handled one by one
    const int full_end = begin + ((end - begin) / N) * N;
    const int stride = blockDim.x * N;
    const uint4 ninf = make_uint4(Vec<T>::NEG_INF, Vec<T>::NEG_INF, Vec<T>::NEG_INF, Vec<T>::NEG_INF);
    // The U loads of the next sweep are issued before the current one is folded,
    // so a thread always has loads in flight; slots past the end read as -inf.
    uint4 cur[U], nxt[U];
    int x = begin + threadIdx.x * N;
#pragma unroll
    for (int u = 0; u < U; ++u)
      cur[u] = (x + u * stride < full_end) ? __ldg(reinterpret_cast<const uint4*>(row + x + u * stride)) : ninf;
    while (x < full_end) {
      const int xn = x + U * stride;
#pragma unroll
      for (int u = 0; u < U; ++u)
        nxt[u] = (xn + u * stride < full_end) ? __ldg(reinterpret_cast<const uint4*>(row + xn + u * stride)) : ninf;
      float v[U][N];
#pragma unroll
      for (int u = 0; u < U; ++u) Vec<T>::convert(cur[u], v[u]);
      if (STATS) fold_stats<U, N, STATS == STAT_SUM>(st, v, x, stride, c);
      if (GUMBEL) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int xu = x + u * stride;
          if ((unsigned)(exclude - xu) < (unsigned)N) {     // the one token left out of the draw
#pragma unroll
            for (int i = 0; i < N; ++i) if (xu + i == exclude) v[u][i] = -CUDART_INF_F;
          }
          if (xu < full_end) fold_gumbel<N>(st, v[u], xu, c, key0, key1, purpose, seq, pos);
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) cur[u] = nxt[u];
      x = xn;
    }
    if (STATS && st.m > -CUDART_INF_F) {
      // settle the arg-max inside its vector: lowest index equal to the maximum
      float vv[N];
      Vec<T>::convert(__ldg(reinterpret_cast<const uint4*>(row + st.idx)), vv);
      int off = 0;
#pragma unroll
      for (int i = N - 1; i >= 0; --i) if (vv[i] == st.m) off = i;
      st.idx += off;
    }
    for (int xt = full_end + threadIdx.x; xt < end; xt += blockDim.x) {
      Stat one = stat_empty();
      fold_one<GUMBEL, STATS>(one, load_logit(row + xt), xt, c, exclude, key0, key1, purpose, seq, pos);
      stat_merge(st, one, c);
    }
  } else {
    for (int xt = begin + threadIdx.x; xt < end; xt += blockDim.x)
      fold_one<GUMBEL, STATS>(st, load_logit(row + xt), xt, c, exclude, key0, key1, purpose, seq, pos);
  }
  return st;
}

__device__ __forceinline__ Stat warp_reduce(Stat st, float c) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    Stat o;
    o.m = __shfl_xor_sync(0xFFFFFFFFu, st.m, off);
    o.s = __shfl_xor_sync(0xFFFFFFFFu, st.s, off);
    o.idx = __shfl_xor_sync(0xFFFFFFFFu, st.idx, off);
    o.gs = __shfl_xor_sync(0xFFFFFFFFu, st.gs, off);
    o.gidx = __shfl_xor_sync(0xFFFFFFFFu, st.gidx, off);
    stat_merge(st, o, c);
  }
  return st;
}

__device__ Stat block_reduce(Stat st, float c) {
  __shared__ Stat sh[SPACE_VERIFY_THREADS / 32];
  st = warp_reduce(st, c);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  if (l == 0) sh[w] = st;
  __syncthreads();
  if (w == 0) {
    st = (l < (int)(blockDim.x >> 5)) ? sh[l] : stat_empty();
    st = warp_reduce(st, c);
  }
  return st;           // valid in warp 0
}


// Reductions for (max, sum, arg-max) only: the maximum (lowest index on ties)
// first, then every contributor rescales its sum once and the sums are added.
// Far fewer exponentials than merging pairwise.
__device__ __forceinline__ void warp_max_idx(float& m, int& idx, int width = 32) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    if (off < width) {
      const float om = __shfl_xor_sync(0xFFFFFFFFu, m, off);
      const int oi = __shfl_xor_sync(0xFFFFFFFFu, idx, off);
      if (om > m || (om == m && oi < idx)) { m = om; idx = oi; }
    }
  }
}
__device__ __forceinline__ float warp_sum(float v, int width = 32) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1)
    if (off < width) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
  return v;
}
// Block-wide (m, s, idx); result valid in thread 0.  gs/gidx are not touched.
__device__ Stat block_reduce_plain(Stat st, float c) {
  __shared__ float sh_m[SPACE_VERIFY_THREADS / 32];
  __shared__ int sh_i[SPACE_VERIFY_THREADS / 32];
  __shared__ float sh_s[SPACE_VERIFY_THREADS / 32];
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  constexpr int NW = SPACE_VERIFY_THREADS / 32;
  float m = st.m; int idx = st.idx;
  warp_max_idx(m, idx);
  if (l == 0) { sh_m[w] = m; sh_i[w] = idx; }
  __syncthreads();
  float bm = sh_m[0]; int bi = sh_i[0];
#pragma unroll
  for (int i = 1; i < NW; ++i) {
    const float om = sh_m[i]; const int oi = sh_i[i];
    if (om > bm || (om == bm && oi < bi)) { bm = om; bi = oi; }
  }
  float sv = (st.m > -CUDART_INF_F) ? st.s * fast_exp2((st.m - bm) * c) : 0.f;
  sv = warp_sum(sv);
  if (l == 0) sh_s[w] = sv;
  __syncthreads();
  Stat r = stat_empty();
  if (threadIdx.x == 0) {
    float tot = 0.f;
#pragma unroll
    for (int i = 0; i < NW; ++i) tot += sh_s[i];
    r.m = bm; r.idx = bi; r.s = tot;
  }
  return r;
}

__device__ __forceinline__ void store_partial(VerifyPartial* p, const Stat& st) {
  VerifyPartial v;
  v.m = st.m; v.s = st.s; v.gs = st.gs; v.idx = st.idx; v.gidx = st.gidx;
  v.pad0 = v.pad1 = v.pad2 = 0;
  *reinterpret_cast<volatile float*>(&p->m) = v.m;
  *reinterpret_cast<volatile float*>(&p->s) = v.s;
  *reinterpret_cast<volatile float*>(&p->gs) = v.gs;
  *reinterpret_cast<volatile int*>(&p->idx) = v.idx;
  *reinterpret_cast<volatile int*>(&p->gidx) = v.gidx;
}

__device__ __forceinline__ Stat load_partial(const VerifyPartial* p) {
  Stat st;
  st.m = __ldcg(&p->m); st.s = __ldcg(&p->s); st.gs = __ldcg(&p->gs);
  st.idx = __ldcg(&p->idx); st.gidx = __ldcg(&p->gidx);
  return st;
}

// Combine the chunk partials of one row with a warp; result valid in every lane.
__device__ Stat gather_row(const VerifyPartial* p, int n_chunks, float c) {
  Stat st = stat_empty();
  for (int i = threadIdx.x & 31; i < n_chunks; i += 32) stat_merge(st, load_partial(p + i), c);
  return warp_reduce(st, c);
}

// Returns true in exactly one block per sequence: the last one to arrive.
__device__ bool arrive_last(int* counter, int expected) {
  __shared__ int last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const int prev = atomicAdd(counter, 1);
    last = (prev == expected - 1);
    if (last) *counter = 0;            // ready for the next launch
  }
  __syncthreads();
  if (last) __threadfence();
  return last != 0;
}

template <typename T, bool VECTOR>
__global__ void __launch_bounds__(SPACE_VERIFY_THREADS)
verify_target_kernel(const VerifyParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.z, t = blockIdx.y, ch = blockIdx.x;
  const int k1 = p.k + 1;
  const T* row = reinterpret_cast<const T*>(p.logits) + ((int64_t)b * p.n_q + (int64_t)t * k1) * p.row_stride;
  const int begin = ch * p.chunk, end = min(p.V, begin + p.chunk);
  Stat st = scan_chunk<T, VECTOR, false, STAT_SUM>(row, begin, end, p.c_t, -1, 0, 0, 0, 0, 0);
  st = block_reduce_plain(st, p.c_t);
  VerifyPartial* part = p.part + ((int64_t)b * (p.k + 2) + t) * p.n_chunks;
  if (threadIdx.x == 0) store_partial(part + ch, st);
  if (!arrive_last(p.counter_a + b, k1 * p.n_chunks)) return;

  // ---- last block of sequence b: acceptance loop of Algorithm 1 ----------
  // Warp tt combines the chunk results of target row tt and evaluates the
  // acceptance test of candidate c_{tt+1}; thread 0 then walks the prefix.
  __shared__ int sh_ok[SPACE_MAX_K + 1];
  __shared__ int sh_bits;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) sh_bits = 0;
  __syncthreads();
  if (warp < k1) {
    const int tt = warp;
    const Stat r = gather_row(part - (int64_t)t * p.n_chunks + (int64_t)tt * p.n_chunks, p.n_chunks, p.c_t);
    if (lane == 0) {
      VerifyRow vr; vr.m = r.m; vr.s = r.s; vr.idx = r.idx; vr.pad = 0;
      p.rows[b * k1 + tt] = vr;
      bool ok = false;
      if (tt < p.k) {                  // row tt scores candidate c_{tt+1}
        const int c = p.cand[b * p.k + tt];
        const bool in_range = (c >= 0 && c < p.V);
        if (!in_range) atomicOr(&sh_bits, SPACE_ST_BAD_CANDIDATE);
        if (p.mode == SPACE_MODE_GREEDY) {
          ok = in_range && (c == r.idx);
        } else {
          const T* base = reinterpret_cast<const T*>(p.logits) + (int64_t)b * p.n_q * p.row_stride;
          const uint32_t seq = p.seq_id ? p.seq_id[b] : (uint32_t)b;
          const int L = p.kv_len ? p.kv_len[b] : 0;
          float q = 0.f;
          if (in_range) {
            const float zc = load_logit(base + (int64_t)tt * k1 * p.row_stride + c);
            q = fast_exp2((zc - r.m) * p.c_t) / r.s;
          }
          const Philox4 w = philox4x32_10(0u, PURPOSE_ACCEPT, seq, (uint32_t)(L + tt + 1), p.key0, p.key1);
          const float pc = p.cand_prob[b * p.k + tt];
          const float lhs = uniform_open(w.x) * pc;                          // r <= Q/P_c  <=>  r*P_c <= Q
          ok = in_range && pc > 0.f && lhs <= q;                             // NaN, zero or negative P_c: rejected
        }
      }
      sh_ok[tt] = ok;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int i_star = 0;
    while (i_star < p.k && sh_ok[i_star]) ++i_star;
    p.n_accept[b] = i_star;
    if (p.status && sh_bits) atomicOr(p.status + b, sh_bits);
  }
}

template <typename T, bool VECTOR>
__global__ void __launch_bounds__(SPACE_VERIFY_THREADS, 3)   // 80 registers, no spills: three blocks per SM
verify_emit_kernel(const VerifyParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const int k1 = p.k + 1;
  const bool sample = p.mode == SPACE_MODE_SAMPLE;
  // One-dimensional grid.  In sampling mode the first B * n_chunks_g blocks are the chunks of the
  // extra-token rows: a logit there costs a Philox block and two logarithms, several times a plain
  // one, so those rows are cut finer (their work spreads over every SM) and start first (no long
  // block is left for the tail of the launch).  Then the mask rows: chunk, sequence, slot.
  const int n_g = sample ? p.B * p.n_chunks_g : 0;
  int b, ch, slot, chunk_len, n_ch;
  if ((int)blockIdx.x < n_g) {
    slot = p.k; b = blockIdx.x / p.n_chunks_g; ch = blockIdx.x - b * p.n_chunks_g;
    chunk_len = p.chunk_g; n_ch = p.n_chunks_g;
  } else {
    int r = blockIdx.x - n_g;
    ch = r % p.n_chunks; r /= p.n_chunks;
    b = r % p.B; slot = r / p.B;
    chunk_len = p.chunk; n_ch = p.n_chunks;
  }
  const int i_star = p.n_accept[b];
  const bool literal = sample && p.resample == SPACE_RESAMPLE_PAPER_LITERAL;
  const int blocks_per_seq = p.k * p.n_chunks + (sample ? p.n_chunks_g : 0);
  const int part_id = (slot == p.k) ? ch : (sample ? p.n_chunks_g : 0) + slot * p.n_chunks + ch;
  const uint32_t seq = p.seq_id ? p.seq_id[b] : (uint32_t)b;
  const int L = p.kv_len ? p.kv_len[b] : 0;
  const T* base = reinterpret_cast<const T*>(p.logits) + (int64_t)b * p.n_q * p.row_stride;
  // With the commit on board every block of the sequence moves its slice of the accepted
  // rows (i* is known to all of them); the last block writes the new length and the tables.
  int Lc = 0;
  if (p.do_commit) {
    Lc = p.cm.kv_len[b];
    if (commit_fits(p.cm, Lc))
      commit_rows(p.cm, b, Lc, max(0, min(i_star, p.k)), part_id, blocks_per_seq, threadIdx.x, blockDim.x);
  }
  // slot o < k: mask row (i*, o+1); slot k: target row i* (extra token, sampling)
  const int brow = (slot < p.k) ? i_star * k1 + slot + 1 : i_star * k1;
  const T* row = base + (int64_t)brow * p.row_stride;
  const int begin = ch * chunk_len, end = min(p.V, begin + chunk_len);
  const float c = sample ? p.c_t : 1.4426950408889634f;
  Stat st;
  if (slot == p.k) {
    int exclude = -1;
    // residual of a point-mass draft (P_c = 1): the rejected token is removed.  A candidate
    // with any other P_c (Algorithm 1 starts from P_c = +inf) was no point mass: a ~ Q.
    if (!literal && i_star < p.k && p.cand_prob[b * p.k + i_star] == 1.0f) exclude = p.cand[b * p.k + i_star];
    // the extra token needs the noisy arg-max alone: the row's sums are known
    st = scan_chunk<T, VECTOR, true, STAT_NONE>(row, begin, end, c, exclude, p.key0, p.key1, PURPOSE_TOKEN,
                                            seq, (uint32_t)(L + i_star + 1));
  } else if (literal) {
    st = scan_chunk<T, VECTOR, true, STAT_SUM>(row, begin, end, c, -1, p.key0, p.key1, PURPOSE_DRAFT, seq,
                                           (uint32_t)(L + i_star + 1 + slot + 1));
  } else if (sample) {
    // point-mass drafts: the new candidates are the rows' arg-maxes with P_c = 1, no sums needed
    st = scan_chunk<T, VECTOR, false, STAT_MAX>(row, begin, end, c, -1, 0, 0, 0, 0, 0);
  } else {
    st = scan_chunk<T, VECTOR, false, STAT_SUM>(row, begin, end, c, -1, 0, 0, 0, 0, 0);
  }
  st = block_reduce(st, c);
  // (chunk results of the emit kernel: SPACE_VERIFY_MAX_CHUNKS slots per row, whatever its cut)
  VerifyPartial* part = p.part + ((int64_t)b * (p.k + 2) + slot) * SPACE_VERIFY_MAX_CHUNKS;
  if (threadIdx.x == 0) store_partial(part + ch, st);
  if (!arrive_last(p.counter_b + b, blocks_per_seq)) return;

  // ---- last block of sequence b: emitted tokens and new candidates -------
  // Warp o combines mask row o (next candidate o+1); warp k the extra-token row.
  __shared__ int sh_bonus;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  VerifyPartial* pb = p.part + (int64_t)b * (p.k + 2) * SPACE_VERIFY_MAX_CHUNKS;
  if (warp < p.k) {
    const int o = warp;
    const Stat r = gather_row(pb + (int64_t)o * SPACE_VERIFY_MAX_CHUNKS, p.n_chunks, c);
    if (lane == 0) {
      int tok; float pr;
      if (!sample)      { tok = r.idx;  pr = 1.f / r.s; }          // softmax at T = 1 of its own maximum
      else if (!literal){ tok = r.idx;  pr = 1.f; }                 // point-mass draft
      else {
        tok = r.gidx;
        const float z = load_logit(base + (int64_t)(i_star * k1 + o + 1) * p.row_stride + tok);
        pr = fast_exp2((z - r.m) * c) / r.s;
      }
      p.next_cand[b * p.k + o] = tok;
      p.next_cand_prob[b * p.k + o] = pr;
    }
  } else if (warp == p.k) {
    int bonus;
    if (sample) bonus = gather_row(pb + (int64_t)p.k * SPACE_VERIFY_MAX_CHUNKS, p.n_chunks_g, c).gidx;
    else bonus = p.rows[b * k1 + i_star].idx;
    if (lane == 0) sh_bonus = bonus;
  }
  __syncthreads();
  if (threadIdx.x < k1) {
    const int j = threadIdx.x;
    int tok = (j < i_star) ? p.cand[b * p.k + j] : (j == i_star ? sh_bonus : -1);
    // <EOS>: keep the tokens before the first one
    const bool is_eos = p.eos_id >= 0 && j <= i_star && tok == p.eos_id;
    const unsigned eos_mask = __ballot_sync((1u << k1) - 1u, is_eos);
    const int first = eos_mask ? __ffs(eos_mask) - 1 : k1;
    const int n_out = eos_mask ? first : i_star + 1;
    p.out_tokens[b * k1 + j] = (j < n_out) ? tok : -1;
    if (j == 0) {
      p.n_out[b] = n_out;
      p.finished[b] = (uint8_t)(eos_mask != 0);
      // every block of the sequence has read the old length by now (arrival counter)
      if (p.do_commit) commit_tables(p.cm, b, Lc, max(0, min(i_star, p.k)), commit_fits(p.cm, Lc));
    }
  }
}



// One launch for greedy mode on small inputs: statistics of every block row,
// then acceptance, emission and next candidates by the last block of a sequence.
// Optional per-block timeline of the single-launch kernel (compiled in with -DSPACE_TIMELINE, as in
// attn_tc.cu): entry, dependency wait returned, logits in registers, counted in, (finishing block) rows
// reduced, done.  Written by thread 0.
#ifdef SPACE_TIMELINE
__device__ unsigned long long g_timeline_verify[4096 * 8];
#define TLV(i) do { const int b_ = (blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x; \
                    if (threadIdx.x == 0 && b_ < 4096) { unsigned long long t_; \
                    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); g_timeline_verify[b_ * 8 + (i)] = t_; } } while (0)
#else
#define TLV(i) do { } while (0)
#endif

// PAGED: the commit on board goes through a page table (a build of its own: the table look-ups are
// not compiled into the contiguous form, whose addressing sits in the critical path).
template <typename T, bool VECTOR, bool PAGED = false>
__global__ void __launch_bounds__(SPACE_VERIFY_THREADS)
verify_fused_kernel(const VerifyParams p, VerifyPartial* fpart) {
  TLV(0);
  pdl_launch_dependents();
  const int b = blockIdx.z, row_i = blockIdx.y, ch = blockIdx.x;
  const int k1 = p.k + 1;
  constexpr float C1 = 1.4426950408889634f;                 // T = 1
  const T* row = reinterpret_cast<const T*>(p.logits) + ((int64_t)b * p.n_q + row_i) * p.row_stride;
  const int begin = ch * p.chunk, end = min(p.V, begin + p.chunk);
  pdl_wait();
  TLV(1);
  int Lc = 0;
  if (p.do_commit) Lc = p.cm.kv_len[b];                     // in flight during the scan
  // (the candidates too: the block that finishes the sequence must not start a memory round trip for them)
  const int my_cand = threadIdx.x < p.k ? p.cand[b * p.k + threadIdx.x] : 0;
  Stat st = scan_chunk<T, VECTOR, false, STAT_SUM>(row, begin, end, C1, -1, 0, 0, 0, 0, 0);
#ifdef SPACE_TIMELINE
  if (st.m != 12345.f) TLV(2);                              // (a use of the result: the stamp follows the loads)
#endif
  // KV commit on board: which candidates are accepted is known only to the last block, at the very
  // end, so every block moves its slice of ALL k candidate rows now, while the logits stream.
  // Rows L+1 .. L+i* end up exactly as the plain commit leaves them; rows L+i*+1 .. L+k, which lie
  // beyond the new length and held mask-token rows nobody reads again, receive the rejected
  // candidates' rows instead.
  if (p.do_commit && commit_fits(p.cm, Lc))
    commit_rows_impl<PAGED>(p.cm, b, Lc, p.k, row_i * p.n_chunks + ch, p.n_q * p.n_chunks, threadIdx.x, blockDim.x);
  // ---- block result and arrival: two block barriers in all.  Every warp reduces its own
  // (maximum, arg-max, sum); eight lanes of warp 0 combine the warps, and lane 0 publishes the
  // chunk's result, fences it and counts the block in.
  constexpr int NW = SPACE_VERIFY_THREADS / 32;
  __shared__ float wm[NW], ws[NW];
  __shared__ int wi[NW];
  __shared__ int sh_last;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  {
    float m = st.m; int idx = st.idx;
    warp_max_idx(m, idx);
    float sv = (st.m > -CUDART_INF_F) ? st.s * fast_exp2((st.m - m) * C1) : 0.f;
    sv = warp_sum(sv);
    if (lane == 0) { wm[warp] = m; wi[warp] = idx; ws[warp] = sv; }
  }
  __syncthreads();
  VerifyPartial* pb = fpart + (int64_t)b * SPACE_MAX_ROWS * SPACE_FUSED_MAX_CHUNKS;
  if (warp == 0) {
    float m = lane < NW ? wm[lane] : -CUDART_INF_F;
    int idx = lane < NW ? wi[lane] : 0x7FFFFFFF;
    const float own = m;
    warp_max_idx(m, idx, NW);
    float sv = (lane < NW && own > -CUDART_INF_F) ? ws[lane] * fast_exp2((own - m) * C1) : 0.f;
    sv = warp_sum(sv, NW);
    if (lane == 0) {
      Stat r = stat_empty();
      r.m = m; r.idx = idx; r.s = sv;
      store_partial(pb + row_i * p.n_chunks + ch, r);
      __threadfence();
      const int prev = atomicAdd(p.counter_a + b, 1);
      const int last = prev == p.n_q * p.n_chunks - 1;
      if (last) p.counter_a[b] = 0;                         // ready for the next launch
      sh_last = last;
    }
  }
  __syncthreads();                                          // (also: every thread's read of the old length precedes the arrival)
  TLV(3);
  if (!sh_last) return;
  // (No fence on this side: every chunk result was fenced by its writer before that block's count, the
  // counts are ordered in L2, and the loads below go to L2 -- after the barrier that followed lane 0's own
  // count.  A fence here would also wait for this thread's row stores of the commit.)

  // ---- last block of sequence b -------------------------------------------
  __shared__ float row_s[SPACE_MAX_ROWS];
  __shared__ int row_idx[SPACE_MAX_ROWS];
  __shared__ int sh_cand[SPACE_MAX_K];
  if (threadIdx.x < p.k) sh_cand[threadIdx.x] = my_cand;
  // two rows per warp at a time: lanes 0..15 and 16..31 each fetch and reduce one row's chunk results
  // (all fetches of a warp are in flight together)
  constexpr int RPW = (SPACE_MAX_ROWS + 2 * NW - 1) / (2 * NW);   // row pairs per warp at most
  float pm[RPW], ps[RPW]; int pi[RPW];
  const int cl = lane & 15;
#pragma unroll
  for (int it = 0; it < RPW; ++it) {
    const int r = (warp + it * NW) * 2 + (lane >> 4);
    pm[it] = -CUDART_INF_F; ps[it] = 0.f; pi[it] = 0x7FFFFFFF;
    if (r < p.n_q && cl < p.n_chunks) {
      const VerifyPartial* q = pb + r * p.n_chunks + cl;
      pm[it] = __ldcg(&q->m); ps[it] = __ldcg(&q->s); pi[it] = __ldcg(&q->idx);
    }
  }
#pragma unroll
  for (int it = 0; it < RPW; ++it) {
    const int r = (warp + it * NW) * 2 + (lane >> 4);
    float bm = pm[it]; int bi = pi[it];
    warp_max_idx(bm, bi, 16);
    float sv = (pm[it] > -CUDART_INF_F) ? ps[it] * fast_exp2((pm[it] - bm) * C1) : 0.f;
    sv = warp_sum(sv, 16);
    if (cl == 0 && r < p.n_q) { row_s[r] = sv; row_idx[r] = bi; }
  }
  __syncthreads();
  TLV(4);
  if (threadIdx.x >= 32) return;
  // acceptance: longest prefix of candidates equal to the arg-max chain
  int i_star = 0, bits = 0;
  for (int t = 0; t < p.k; ++t) {
    const int c = sh_cand[t];
    if (c < 0 || c >= p.V) bits |= SPACE_ST_BAD_CANDIDATE;
  }
  while (i_star < p.k && sh_cand[i_star] >= 0 && sh_cand[i_star] < p.V &&
         sh_cand[i_star] == row_idx[i_star * k1]) ++i_star;
  const int j = lane;
  if (j < k1) {
    int tok = (j < i_star) ? sh_cand[j] : (j == i_star ? row_idx[i_star * k1] : -1);
    const bool is_eos = p.eos_id >= 0 && j <= i_star && tok == p.eos_id;
    const unsigned eos_mask = __ballot_sync((1u << k1) - 1u, is_eos);
    const int n_out = eos_mask ? __ffs(eos_mask) - 1 : i_star + 1;
    p.out_tokens[b * k1 + j] = (j < n_out) ? tok : -1;
    if (j < p.k) {                                          // next candidate j+1 from mask row (i*, j+1)
      const int mr = i_star * k1 + j + 1;
      p.next_cand[b * p.k + j] = row_idx[mr];
      p.next_cand_prob[b * p.k + j] = 1.f / row_s[mr];      // softmax at T = 1 of its own maximum
    }
    if (j == 0) {
      p.n_accept[b] = i_star;
      p.n_out[b] = n_out;
      p.finished[b] = (uint8_t)(eos_mask != 0);
      if (p.status && bits) atomicOr(p.status + b, bits);
      // new length and index tables; every block of the sequence read the old length before it arrived
      if (p.do_commit) commit_tables(p.cm, b, Lc, i_star, commit_fits(p.cm, Lc));
      TLV(5);
    }
  }
}

template <typename T, bool VECTOR>
void launch_fused(space_ctx* ctx, const VerifyParams& p, cudaStream_t st) {
  ProfScope ps(ctx, SPACE_K_VERIFY_TARGET, st);
  if (p.do_commit && p.cm.page_table)
    launch_pdl(verify_fused_kernel<T, VECTOR, true>, dim3(p.n_chunks, p.n_q, p.B), dim3(SPACE_VERIFY_THREADS), 0, st, p, ctx->vfused);
  else
  launch_pdl(verify_fused_kernel<T, VECTOR>, dim3(p.n_chunks, p.n_q, p.B), dim3(SPACE_VERIFY_THREADS), 0, st, p, ctx->vfused);
}

template <typename T, bool VECTOR>
void launch_both(space_ctx* ctx, const VerifyParams& p, int n_slots_b, cudaStream_t st) {
  dim3 ga(p.n_chunks, p.k + 1, p.B);
  const dim3 gb(p.B * (p.k * p.n_chunks + (p.mode == SPACE_MODE_SAMPLE ? p.n_chunks_g : 0)));
  {
    ProfScope ps(ctx, SPACE_K_VERIFY_TARGET, st);
    launch_pdl(verify_target_kernel<T, VECTOR>, ga, dim3(SPACE_VERIFY_THREADS), 0, st, p);
  }
  {
    ProfScope ps(ctx, SPACE_K_VERIFY_EMIT, st);
    launch_pdl(verify_emit_kernel<T, VECTOR>, gb, dim3(SPACE_VERIFY_THREADS), 0, st, p);
  }
}

__global__ void philox_debug_kernel(uint32_t k0, uint32_t k1, int64_t n, const uint32_t* c0,
                                    const uint32_t* c1, const uint32_t* c2, const uint32_t* c3,
                                    uint32_t* out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const Philox4 r = philox4x32_10(c0[i], c1[i], c2[i], c3[i], k0, k1);
  out[4 * i] = r.x; out[4 * i + 1] = r.y; out[4 * i + 2] = r.z; out[4 * i + 3] = r.w;
}

}  // namespace

#ifdef SPACE_TIMELINE
extern "C" int space_debug_timeline_read_verify(unsigned long long* host_dst, int n_blocks) {
  return cuda_ok(cudaMemcpyFromSymbol(host_dst, g_timeline_verify, sizeof(unsigned long long) * 8 * n_blocks));
}
#endif

int launch_verify(space_ctx* ctx, const space_verify_args* a, const space_commit_args* cm, cudaStream_t st) {
  if (a->mode == SPACE_MODE_SAMPLE && a->top_k > 0) {
    // filtered target distributions: kernels of their own (verify_filter.cu); the commit follows as its own launch
    const int rc = launch_verify_filtered(ctx, a, st);
    if (rc != SPACE_OK || !cm) return rc;
    return launch_commit(ctx, cm, st);
  }
  if (cm && cm->page_table) {
    // paged cache: only the single-launch greedy form carries the commit through a page table; the
    // two-launch form is followed by the commit kernel
    const int64_t all_b = (int64_t)a->batch * (a->k + 1) * (a->k + 1) * a->vocab * (a->logits_dtype == SPACE_DTYPE_F32 ? 4 : 2);
    if (!(a->mode == SPACE_MODE_GREEDY && all_b <= SPACE_FUSED_MAX_BYTES)) {
      const int rc = launch_verify(ctx, a, nullptr, st);
      if (rc != SPACE_OK) return rc;
      return launch_commit(ctx, cm, st);
    }
  }
  VerifyParams p;
  p.do_commit = cm != nullptr;
  if (cm) fill_commit_params(ctx, cm, &p.cm); else memset(&p.cm, 0, sizeof(p.cm));
  p.B = a->batch; p.k = a->k; p.V = a->vocab; p.n_q = (a->k + 1) * (a->k + 1);
  p.mode = a->mode; p.resample = a->resample; p.eos_id = a->eos_id;
  const float T = (a->mode == SPACE_MODE_SAMPLE) ? a->temperature : 1.0f;
  p.c_t = 1.4426950408889634f / T;
  p.inv_t = 1.0f / T;
  p.key0 = (uint32_t)(a->seed & 0xFFFFFFFFull); p.key1 = (uint32_t)(a->seed >> 32);
  p.logits = a->logits; p.row_stride = a->logits_row_stride;
  p.cand = a->cand; p.cand_prob = a->cand_prob; p.seq_id = a->seq_id; p.kv_len = a->kv_len;
  p.n_accept = a->n_accept; p.out_tokens = a->out_tokens; p.n_out = a->n_out;
  p.next_cand = a->next_cand; p.next_cand_prob = a->next_cand_prob; p.finished = a->finished;
  p.status = a->status;
  p.part = ctx->vpart; p.rows = ctx->vrow;
  p.counter_a = ctx->counters; p.counter_b = ctx->counters + ctx->cfg.max_batch;

  const int esz = a->logits_dtype == SPACE_DTYPE_F32 ? 4 : 2;
  const int vec = 16 / esz;
  const bool vector = ((uintptr_t)a->logits % 16 == 0) && ((a->logits_row_stride * esz) % 16 == 0);
  // small greedy problem: one launch over all block rows (see the file header)
  const int64_t all_bytes = (int64_t)a->batch * p.n_q * a->vocab * esz;
  if (a->mode == SPACE_MODE_GREEDY && all_bytes <= SPACE_FUSED_MAX_BYTES) {
    const int rows_all = a->batch * p.n_q;
    int nc = ctx->sm_count / rows_all;                      // about one block per SM: few arrivals, four loads in flight
    const int min_chunk = SPACE_VERIFY_THREADS * vec;
    const int max_nc = (a->vocab + min_chunk - 1) / min_chunk;
    if (nc > max_nc) nc = max_nc;
    if (nc > SPACE_FUSED_MAX_CHUNKS) nc = SPACE_FUSED_MAX_CHUNKS;
    if (nc < 1) nc = 1;
    int chunk = (a->vocab + nc - 1) / nc;
    chunk = ((chunk + vec - 1) / vec) * vec;
    nc = (a->vocab + chunk - 1) / chunk;
    p.n_chunks = nc; p.chunk = chunk; p.n_chunks_g = 0; p.chunk_g = 0;
    if (a->logits_dtype == SPACE_DTYPE_F32) {
      if (vector) launch_fused<float, true>(ctx, p, st); else launch_fused<float, false>(ctx, p, st);
    } else {
      if (vector) launch_fused<__nv_bfloat16, true>(ctx, p, st); else launch_fused<__nv_bfloat16, false>(ctx, p, st);
    }
    ctx->launches += 1;
    return cuda_ok(cudaGetLastError());
  }
  // enough chunks to put about four blocks on every SM: little more than one resident
  // wave (measured on the 64-sequence sampling workload: 4 per SM 29 / 39 us, 8 per SM
  // 31 / 43 us, 16 per SM 38 / 54 us), but no chunk below four sweeps of a block
  const int rows = a->batch * (a->k + 1);
  int nc = (4 * ctx->sm_count + rows - 1) / rows;
  const int min_chunk = SPACE_VERIFY_THREADS * vec * 4;
  const int max_nc = (a->vocab + min_chunk - 1) / min_chunk;
  if (nc > max_nc) nc = max_nc;
  if (nc > SPACE_VERIFY_MAX_CHUNKS) nc = SPACE_VERIFY_MAX_CHUNKS;
  if (nc < 1) nc = 1;
  int chunk = (a->vocab + nc - 1) / nc;
  chunk = ((chunk + vec - 1) / vec) * vec;
  nc = (a->vocab + chunk - 1) / chunk;
  p.n_chunks = nc; p.chunk = chunk;
  const int n_slots_b = (a->mode == SPACE_MODE_SAMPLE) ? a->k + 1 : a->k;
  // the extra-token row has a cut of its own (its logits cost several times a plain row's)
  {
    int ncg = nc;                                           // (measured: a finer cut of this row, up to 8x, is no faster)
    const int min_chunk_g = SPACE_VERIFY_THREADS * vec * 4;
    const int max_ncg = (a->vocab + min_chunk_g - 1) / min_chunk_g;
    if (ncg > max_ncg) ncg = max_ncg;
    if (ncg > SPACE_VERIFY_MAX_CHUNKS) ncg = SPACE_VERIFY_MAX_CHUNKS;
    if (ncg < 1) ncg = 1;
    int cg = (a->vocab + ncg - 1) / ncg;
    cg = ((cg + vec - 1) / vec) * vec;
    p.n_chunks_g = (a->vocab + cg - 1) / cg; p.chunk_g = cg;
  }

  if (a->logits_dtype == SPACE_DTYPE_F32) {
    if (vector) launch_both<float, true>(ctx, p, n_slots_b, st); else launch_both<float, false>(ctx, p, n_slots_b, st);
  } else {
    if (vector) launch_both<__nv_bfloat16, true>(ctx, p, n_slots_b, st);
    else launch_both<__nv_bfloat16, false>(ctx, p, n_slots_b, st);
  }
  ctx->launches += 2;
  return cuda_ok(cudaGetLastError());
}

int launch_philox_debug(uint64_t seed, int64_t n, const uint32_t* c0, const uint32_t* c1,
                        const uint32_t* c2, const uint32_t* c3, uint32_t* out, cudaStream_t st) {
  if (n <= 0) return SPACE_OK;
  philox_debug_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(
      (uint32_t)(seed & 0xFFFFFFFFull), (uint32_t)(seed >> 32), n, c0, c1, c2, c3, out);
  return cuda_ok(cudaGetLastError());
}

// ---------------------------------------------------------------------------
// Allocation-free greedy verification (space_verify_greedy_noalloc).
//
// The scratch that verify_fused_kernel needs (chunk results and one arrival
// counter per sequence) lives in this file-scope device array instead of a
// context workspace, so the entry point never calls cudaMalloc.  Every GPU that
// loads the library holds the array until the process exits.
#define SPACE_NOALLOC_COUNTER_BYTES 256
#define SPACE_NOALLOC_SCRATCH_BYTES \
  (SPACE_NOALLOC_COUNTER_BYTES +      \
   SPACE_NOALLOC_MAX_BATCH * SPACE_MAX_ROWS * SPACE_FUSED_MAX_CHUNKS * (int)sizeof(VerifyPartial))
static __device__ __align__(256) unsigned char g_noalloc_scratch[SPACE_NOALLOC_SCRATCH_BYTES];

namespace {
constexpr int NOALLOC_MAX_DEVICES = 64;
// The array's name is only a host-side handle; the address kernels can use is
// looked up once per device (with that device current) and kept here.
void* g_noalloc_ptr[NOALLOC_MAX_DEVICES];
int g_noalloc_sms[NOALLOC_MAX_DEVICES];
}  // namespace

int launch_verify_noalloc(const space_verify_args* a, cudaStream_t st) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES) return SPACE_E_NO_DEVICE;
  if (!g_noalloc_ptr[dev]) {
    // first call on this device: resolve the device address of the scratch array
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return SPACE_E_CUDA;
    }
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
      cudaGetLastError();
      return SPACE_E_CUDA;
    }
    // With lazy module loading a kernel's code reaches the device at its first use: ask for the
    // attributes of all four variants now, so that no later call is the one that loads anything.
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, verify_fused_kernel<float, true>) != cudaSuccess ||
        cudaFuncGetAttributes(&fa, verify_fused_kernel<float, false>) != cudaSuccess ||
        cudaFuncGetAttributes(&fa, verify_fused_kernel<__nv_bfloat16, true>) != cudaSuccess ||
        cudaFuncGetAttributes(&fa, verify_fused_kernel<__nv_bfloat16, false>) != cudaSuccess) {
      cudaGetLastError();
      return SPACE_E_CUDA;
    }
    g_noalloc_sms[dev] = sms;
    g_noalloc_ptr[dev] = ptr;
  }
  unsigned char* base = static_cast<unsigned char*>(g_noalloc_ptr[dev]);
  // the arrival counters must start at zero whatever an earlier call left behind
  if (cudaMemsetAsync(base, 0, SPACE_NOALLOC_COUNTER_BYTES, st) != cudaSuccess) return SPACE_E_CUDA;

  VerifyParams p;
  p.B = a->batch; p.k = a->k; p.V = a->vocab; p.n_q = (a->k + 1) * (a->k + 1);
  p.mode = SPACE_MODE_GREEDY; p.resample = SPACE_RESAMPLE_RESIDUAL_POINTMASS; p.eos_id = a->eos_id;
  p.c_t = 1.4426950408889634f; p.inv_t = 1.0f;
  p.key0 = 0; p.key1 = 0;
  p.logits = a->logits; p.row_stride = a->logits_row_stride;
  p.cand = a->cand; p.cand_prob = a->cand_prob; p.seq_id = a->seq_id; p.kv_len = a->kv_len;
  p.n_accept = a->n_accept; p.out_tokens = a->out_tokens; p.n_out = a->n_out;
  p.next_cand = a->next_cand; p.next_cand_prob = a->next_cand_prob; p.finished = a->finished;
  p.status = a->status;
  p.part = nullptr; p.rows = nullptr;
  p.counter_a = reinterpret_cast<int*>(base); p.counter_b = nullptr;
  p.do_commit = 0; memset(&p.cm, 0, sizeof(p.cm));
  VerifyPartial* fpart = reinterpret_cast<VerifyPartial*>(base + SPACE_NOALLOC_COUNTER_BYTES);

  const int esz = a->logits_dtype == SPACE_DTYPE_F32 ? 4 : 2;
  const int vec = 16 / esz;
  const bool vector = ((uintptr_t)a->logits % 16 == 0) && ((a->logits_row_stride * esz) % 16 == 0);
  const int rows_all = a->batch * p.n_q;
  int nc = g_noalloc_sms[dev] / rows_all;
  const int min_chunk = SPACE_VERIFY_THREADS * vec;
  const int max_nc = (a->vocab + min_chunk - 1) / min_chunk;
  if (nc > max_nc) nc = max_nc;
  if (nc > SPACE_FUSED_MAX_CHUNKS) nc = SPACE_FUSED_MAX_CHUNKS;
  if (nc < 1) nc = 1;
  int chunk = (a->vocab + nc - 1) / nc;
  chunk = ((chunk + vec - 1) / vec) * vec;
  nc = (a->vocab + chunk - 1) / chunk;
  p.n_chunks = nc; p.chunk = chunk;
  const dim3 grid(nc, p.n_q, a->batch), block(SPACE_VERIFY_THREADS);
  cudaError_t e;
  if (a->logits_dtype == SPACE_DTYPE_F32) {
    e = vector ? launch_pdl(verify_fused_kernel<float, true>, grid, block, 0, st, p, fpart)
               : launch_pdl(verify_fused_kernel<float, false>, grid, block, 0, st, p, fpart);
  } else {
    e = vector ? launch_pdl(verify_fused_kernel<__nv_bfloat16, true>, grid, block, 0, st, p, fpart)
               : launch_pdl(verify_fused_kernel<__nv_bfloat16, false>, grid, block, 0, st, p, fpart);
  }
  return cuda_ok(e);
}
