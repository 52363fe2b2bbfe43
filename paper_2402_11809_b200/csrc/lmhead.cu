// Output projection fused with greedy verification (Algorithm 1: the end of the
// model call P = M(I) and the loop after it).
//
// logits[r, x] = <h_r, W_x> for the (k+1)^2 block rows of every sequence and the
// whole vocabulary, but the logits never reach memory: the product runs on the
// tensor cores with the block rows on the MMA M extent (A = hidden rows, K-major)
// and up to 256 tokens on the N extent (B = rows of W, K-major; fp32 accumulators
// in TMEM: lane = block row, column = token).  An instruction of this kind costs
// about the same whatever its N, so the tokens go on N: measured with the tokens
// on M (128 per instruction) the 512 instructions of a thread block took longer
// than its share of W takes to arrive.  Every epilogue thread owns one block row
// and folds its accumulator columns into (max, lowest arg-max, sum exp(z - max))
// in registers, without any exchange between threads.  The last thread block to
// finish combines the vocabulary ranges and runs the acceptance scan, the extra
// token, the <EOS> cut and the next candidates.
//
// The output embedding is streamed exactly once (the step's HBM roof); the
// hidden rows are re-read from L2 by every thread block.
//
// Vocabulary ranges: thread block c owns rows [V*c/G, V*(c+1)/G) and covers them
// with boxes of n_box rows (256, or the longest range rounded up to 16 when that
// is shorter); the last box of a range is loaded through a second tensor map
// whose box holds only the rows a range's tail can have, so a range reads at
// most 15 rows of its neighbour.
//
// Warps: 0 TMA producer, 1 TMEM owner and MMA issuer, 2..5 epilogue (one TMEM
// lane quarter each).  With at most 128 block rows two accumulators alternate
// between boxes so that the epilogue of one box runs under the products of the
// next.  Every wait is bounded; an expired wait sets SPACE_ST_TIMEOUT, the block
// drains and exits.
#include "common.cuh"
#include "tc_common.cuh"
#include <cuda.h>
#include <math_constants.h>

namespace {

constexpr int LM_THREADS = 192;
constexpr int LM_M = 128;                   // block rows per accumulator (MMA M)
constexpr int LM_MAX_BOX = 256;             // vocabulary rows per box (MMA N), at most
constexpr int LM_KB = 64;                   // hidden elements per slice (128 bytes: one swizzle row)
constexpr int LM_MAX_STAGES = 10;
constexpr float LM_NEG = -3.0e38f;          // "no logit yet": finite, so that differences never give NaN
constexpr int LM_MAX_N = 256;               // block rows of the whole batch, padded to 16
constexpr uint64_t LM_WAIT_NS = 1000000000ull;
constexpr float LOG2E = 1.4426950408889634f;

struct LmPartial { float m, s; int idx, pad; };   // 16 bytes
struct LmNoisy { float gs, gz; int gidx, pad; };   // best noisy score of a range, the logit that has it, its token

struct LmParams {
  CUtensorMap tm_w, tm_wt, tm_h;   // W in boxes of n_box rows, W in boxes of tail_rows rows, hidden rows
  int B, k, V, D, n_q;
  int n_rows;                 // B * n_q
  int n_pad;                  // n_rows rounded up to 16: rows of the hidden-state tile
  int n_mt;                   // accumulators of 128 block rows (1 or 2)
  int stages;
  int n_box;                  // rows of the first tensor map's box (N of its products)
  int tail_rows;              // rows of the second tensor map's box
  int kbs;                    // 64-element slices of the hidden dimension per stage
  int eos_id;
  int mode, resample;         // SPACE_MODE_*, SPACE_RESAMPLE_*
  float c_t;                  // log2(e) / T: exponent scale of the sums and of the noisy scores (sampling)
  uint32_t key0, key1;        // Philox key
  uint32_t seq_base;          // sequence id of the group's first sequence when seq_id is NULL
  const float* cand_prob; const uint32_t* seq_id; const int32_t* kv_len;
  LmNoisy* gpart;             // [n_rows][gridDim.x] (sampling)
  float* zc;                  // [n_rows] logit of the candidate a target row scores, written by the block that owns the token
  const int32_t* cand;
  int32_t* n_accept; int32_t* out_tokens; int32_t* n_out; int32_t* next_cand;
  float* next_cand_prob; uint8_t* finished; int32_t* status;
  float* row_max; int32_t* row_argmax;
  LmPartial* part;            // [n_rows][gridDim.x]
  unsigned long long* keys;   // [n_rows] arg-max keys, combined with atomicMax; zero between launches
  int* counter;               // arrival counter (self-resetting)
  int* err;
};

// PTX helpers: tc_common.cuh.  Every wait of this kernel is bounded by LM_WAIT_NS.
// `backoff`: sleep between polls (the epilogue warps, which wait for a whole group of products).
using namespace tc;
__device__ __noinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* err, int site,
                                          bool backoff = false) {
  return mbar_wait_bounded(bar, parity, abort_flag, err, site, LM_WAIT_NS, backoff ? 128u : 0u);
}
__device__ __noinline__ void mbar_drain(uint32_t bar, uint32_t parity) { mbar_drain_bounded(bar, parity, LM_WAIT_NS); }
// Shared-memory matrix descriptor: K-major rows of 128 bytes, 128-byte swizzle
// (groups of 8 rows 1024 bytes apart), descriptor version of sm_100.
__device__ __forceinline__ uint64_t smem_desc_k128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3FFF);
  d |= (uint64_t)((16u >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((1024u >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// Instruction descriptor: bf16 x bf16 -> f32, M = 128, N = n, both operands K-major.
__device__ __forceinline__ uint32_t instr_desc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(LM_M >> 4) << 24);
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Statistics of a set of logits: (m, s, i) = (max, sum of exp(z - m), lowest arg-max);
// the empty set is (LM_NEG, 0, INT_MAX).  fold: union of two sets.  One of the two
// exponentials is exp(0), so a single ex2 serves.
__device__ __forceinline__ void stat_fold(float& m, float& s, int& i, float m2, float s2, int i2) {
  if (m2 > m || (m2 == m && i2 < i)) i = i2;
  const float e = fast_exp2(-fabsf(m - m2) * LOG2E);
  s = (m >= m2) ? fmaf(s2, e, s) : fmaf(s, e, s2);
  m = fmaxf(m, m2);
}

// (maximum, lowest token) of a row as one 64-bit key whose unsigned order is "larger logit
// first, then lower token": the ranges of all thread blocks combine with one atomicMax each.
// 0 is below every key of a real logit.
__device__ __forceinline__ unsigned long long argmax_key(float m, int idx) {
  uint32_t u = __float_as_uint(m);
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  return ((unsigned long long)u << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)idx);
}
__device__ __forceinline__ void argmax_unkey(unsigned long long key, float& m, int& idx) {
  uint32_t u = (uint32_t)(key >> 32);
  u = (u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u;
  m = __uint_as_float(u);
  idx = (int)(0xFFFFFFFFu - (uint32_t)key);
}

// Fold 16 consecutive tokens x0 .. x0+15 (the first nv of them valid) into a row's statistics.
__device__ __forceinline__ void fold16(float& m, float& s, int& idx, const uint32_t* v, int x0, int nv) {
  float z[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) z[j] = (j < nv) ? __uint_as_float(v[j]) : LM_NEG;
  float cm = z[0];
#pragma unroll
  for (int j = 1; j < 16; ++j) cm = fmaxf(cm, z[j]);
  if (cm > m) {                                           // strictly larger: an earlier token keeps a tie
    int at = 15;
#pragma unroll
    for (int j = 14; j >= 0; --j) at = (z[j] == cm) ? j : at;
    idx = x0 + at;
    s *= fast_exp2((m - cm) * LOG2E);
    m = cm;
  }
  const float ms = -m * LOG2E;
  float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
  for (int j = 0; j < 16; j += 4) {
    a0 += fast_exp2(fmaf(z[j], LOG2E, ms));
    a1 += fast_exp2(fmaf(z[j + 1], LOG2E, ms));
    a2 += fast_exp2(fmaf(z[j + 2], LOG2E, ms));
    a3 += fast_exp2(fmaf(z[j + 3], LOG2E, ms));
  }
  s += (a0 + a1) + (a2 + a3);
}

// What an epilogue thread keeps of one block row in sampling mode.
struct RowNoisy {
  float gs, gz; int gidx;     // best noisy score so far, the logit that has it, its token
  float zc;                   // logit of the candidate this (target) row scores
  int cand_tok;               // that candidate, or -1
  int exclude;                // token left out of the draw (the rejected point-mass candidate), or -1
  uint32_t purpose, seq, pos; // Philox counter words of this row's noise
  bool noisy;                 // this row draws a token at all
};

// Sampling-mode fold of 16 consecutive tokens x0 .. x0+15 (x0 a multiple of 16, the first nv valid):
// (max, lowest arg-max, sum of exp2((z - max) c)), the candidate's own logit when it lies here, and
// the best Gumbel-perturbed score z c + noise(token) -- the noise of token x is lane x & 3 of the
// Philox block with counter word x >> 2, as in the verification kernels.
__device__ __forceinline__ void fold16_noisy(float& m, float& s, int& idx, RowNoisy& r, const uint32_t* v, int x0,
                                             int nv, float c, uint32_t key0, uint32_t key1) {
  float z[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) z[j] = (j < nv) ? __uint_as_float(v[j]) : LM_NEG;
  float cm = z[0];
#pragma unroll
  for (int j = 1; j < 16; ++j) cm = fmaxf(cm, z[j]);
  if (cm > m) {
    int at = 15;
#pragma unroll
    for (int j = 14; j >= 0; --j) at = (z[j] == cm) ? j : at;
    idx = x0 + at;
    s *= fast_exp2((m - cm) * c);
    m = cm;
  }
  const float ms = -m * c;
  float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
  for (int j = 0; j < 16; j += 4) {
    a0 += fast_exp2(fmaf(z[j], c, ms));
    a1 += fast_exp2(fmaf(z[j + 1], c, ms));
    a2 += fast_exp2(fmaf(z[j + 2], c, ms));
    a3 += fast_exp2(fmaf(z[j + 3], c, ms));
  }
  s += (a0 + a1) + (a2 + a3);
  if ((unsigned)(r.cand_tok - x0) < 16u) {
#pragma unroll
    for (int j = 0; j < 16; ++j) if (x0 + j == r.cand_tok) r.zc = z[j];
  }
  if (r.noisy) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const Philox4 ph = philox4x32_10((uint32_t)((x0 >> 2) + i), r.purpose, r.seq, r.pos, key0, key1);
      const uint32_t w[4] = {ph.x, ph.y, ph.z, ph.w};
#pragma unroll
      for (int l = 0; l < 4; ++l) {
        const int j = 4 * i + l;
        const float sc = fmaf(z[j], c, gumbel2_from_uniform(uniform_open(w[l])));
        if (j < nv && x0 + j != r.exclude && sc > r.gs) { r.gs = sc; r.gidx = x0 + j; r.gz = z[j]; }
      }
    }
  }
}

// Per-row constants of the sampling mode: block row `row` of the batch is row i = row mod n_q of
// sequence b; target rows (i = t(k+1)) score candidate c_{t+1} and draw the extra token of the
// case i* = t at position L+t+1; mask rows (t, o) draw candidate o of that case at position
// L+t+1+o when candidates are sampled (Algorithm 1 as printed).
__device__ __forceinline__ void row_noisy_init(RowNoisy& r, const LmParams& p, int row) {
  r.gs = -CUDART_INF_F; r.gz = 0.f; r.gidx = 0x7FFFFFFF; r.zc = LM_NEG;
  r.cand_tok = -1; r.exclude = -1; r.purpose = 0; r.seq = 0; r.pos = 0; r.noisy = false;
  if (row >= p.n_rows) return;
  const int k1 = p.k + 1;
  const int b = row / p.n_q, i = row - b * p.n_q;
  const int t = i / k1, o = i - t * k1;
  const bool literal = p.resample == SPACE_RESAMPLE_PAPER_LITERAL;
  r.seq = p.seq_id ? p.seq_id[b] : p.seq_base + (uint32_t)b;
  const int L = p.kv_len ? p.kv_len[b] : 0;
  if (o == 0) {
    r.noisy = true; r.purpose = PURPOSE_TOKEN; r.pos = (uint32_t)(L + t + 1);
    if (t < p.k) {
      r.cand_tok = p.cand[b * p.k + t];
      if (!literal && p.cand_prob[b * p.k + t] == 1.0f) r.exclude = r.cand_tok;   // residual of a point mass
    }
  } else if (literal) {
    r.noisy = true; r.purpose = PURPOSE_DRAFT; r.pos = (uint32_t)(L + t + 1 + o);
  }
}

// (max, lowest arg-max) over the warp, result in every lane
__device__ __forceinline__ void warp_max_idx(float& m, int& idx) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float om = __shfl_xor_sync(0xFFFFFFFFu, m, off);
    const int oi = __shfl_xor_sync(0xFFFFFFFFu, idx, off);
    if (om > m || (om == m && oi < idx)) { m = om; idx = oi; }
  }
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
  return v;
}

// Shared-memory plan (dynamic, 1024-byte aligned base):
//   [stages]{ [kbs] hidden tiles of n_pad*128 bytes, [kbs] W tiles of n_box*128 bytes } | pad |
//   barriers | row results [n_pad] x 2 | candidates | misc
// A product reads 128 rows from a hidden tile's address whatever n_pad is: the rows past the
// tile are whatever follows in shared memory (the stage's W tiles, then `pad`) and only reach
// accumulator lanes nobody reads.  `pad` keeps that read inside the allocation.
struct LmSmem {
  uint32_t a_bytes, b_bytes, b_in_stage, stage_bytes, bar_off, row_off, cand_off, misc_off, total;
  __host__ __device__ LmSmem(int n_pad, int n_box, int stages, int kbs) {
    a_bytes = (uint32_t)n_pad * LM_KB * 2;
    b_bytes = (uint32_t)n_box * LM_KB * 2;
    b_in_stage = (uint32_t)kbs * a_bytes;
    stage_bytes = b_in_stage + (uint32_t)kbs * b_bytes;
    const uint32_t reach = 16384u * (n_pad > LM_M ? 2u : 1u);            // bytes a product reads from a hidden tile
    const uint32_t have = a_bytes + (uint32_t)kbs * b_bytes;             // bytes that follow the last hidden tile's start
    const uint32_t pad = reach > have ? (reach - have + 1023u) / 1024u * 1024u : 0u;
    bar_off = (uint32_t)stages * stage_bytes + pad;
    row_off = bar_off + 8u * (2 * LM_MAX_STAGES + 4);
    cand_off = row_off + 2u * 4u * (uint32_t)n_pad;                      // candidates of the batch: fewer than n_pad
    misc_off = cand_off + 4u * (uint32_t)n_pad;
    total = misc_off + 64u;
  }
};

__global__ void __launch_bounds__(LM_THREADS, 1) lmhead_verify_kernel(const __grid_constant__ LmParams p) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t sm_base = smem_u32(smem_raw);
  const LmSmem L(p.n_pad, p.n_box, p.stages, p.kbs);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int S = p.stages;
  const uint32_t bar0 = sm_base + L.bar_off;
#define LBAR(i) (bar0 + 8u * (uint32_t)(i))
  const int B_FULL = 0, B_EMPTY = LM_MAX_STAGES, B_ACCFULL = 2 * LM_MAX_STAGES, B_ACCEMPTY = 2 * LM_MAX_STAGES + 2;
  float* row_s = reinterpret_cast<float*>(smem_raw + L.row_off);           // [n_pad]
  int* row_i = reinterpret_cast<int*>(row_s + p.n_pad);
  int* cand_s = reinterpret_cast<int*>(smem_raw + L.cand_off);            // [B * k]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_raw + L.misc_off);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_raw + L.misc_off + 4);
  int* last_flag = reinterpret_cast<int*>(smem_raw + L.misc_off + 8);

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    *abort_flag = (sm_base & 1023u) ? 1 : 0;               // swizzled tiles need a 1024-byte aligned base
    for (int s = 0; s < S; ++s) { mbar_init(LBAR(B_FULL + s), 1); mbar_init(LBAR(B_EMPTY + s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(LBAR(B_ACCFULL + a), 1); mbar_init(LBAR(B_ACCEMPTY + a), 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (warp == 0 && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&p.tm_w) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&p.tm_wt) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&p.tm_h) : "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_wait();                                              // global memory from here on

  // this thread block's vocabulary range and its boxes
  const int G = gridDim.x, c = blockIdx.x;
  // (range boundaries are multiples of 16 tokens, so that a group of 16 accumulator columns
  // always starts on a Philox block)
  const int r0 = (int)(((long long)p.V * c) / G) & ~15;
  const int r1 = (c == G - 1) ? p.V : ((int)(((long long)p.V * (c + 1)) / G) & ~15);
  const int nb = (r1 - r0 + p.n_box - 1) / p.n_box;
  const int KB = (p.D + LM_KB - 1) / LM_KB;
  const int kbs = p.kbs;
  const int n_bufs = p.n_mt == 1 ? 2 : 1;                  // accumulator buffers of n_mt x 256 columns

  if (warp == 0) {
    // ================= producer ==============================================
    if (lane == 0) {
      const int ipb = (KB + kbs - 1) / kbs;                // stages per box
      const uint32_t n_it = (uint32_t)(nb * ipb);
      bool ok = !*abort_flag;
      // stage `it`: the W tiles and the hidden tiles of its slices
      auto issue = [&](uint32_t it) {
        const int box = (int)it / ipb, kb0 = ((int)it - box * ipb) * kbs;
        const int s = it % S;
        const int nk = min(kbs, KB - kb0);
        const int row0 = r0 + box * p.n_box;
        const bool tail = r1 - row0 <= p.tail_rows;        // the remaining rows fit the small box
        const uint32_t st_base = sm_base + (uint32_t)s * L.stage_bytes;
        const CUtensorMap* tm = tail ? &p.tm_wt : &p.tm_w;
        const uint32_t w_bytes = (uint32_t)(tail ? p.tail_rows : p.n_box) * LM_KB * 2;
        mbar_expect_tx(LBAR(B_FULL + s), (uint32_t)nk * (w_bytes + L.a_bytes));
        for (int j = 0; j < nk; ++j)
          tma_load_4d(st_base + L.b_in_stage + (uint32_t)j * L.b_bytes, tm, LBAR(B_FULL + s), (kb0 + j) * LM_KB, row0, 0, 0);
        for (int j = 0; j < nk; ++j)
          tma_load_4d(st_base + (uint32_t)j * L.a_bytes, &p.tm_h, LBAR(B_FULL + s), (kb0 + j) * LM_KB, 0, 0, 0);
      };
      // (requesting the first stages' W tiles before the dependency wait, so that they stream under the
      // previous kernel's tail, measured 0.8 us slower per step in graph replay and was left out)
      uint32_t it = 0;
      for (; it < n_it && ok; ++it) {
        if (it >= (uint32_t)S) ok = mbar_wait(LBAR(B_EMPTY + it % S), ((it / S) - 1) & 1, abort_flag, p.err, 1);
        if (!ok) break;
        issue(it);
      }
      if (!ok) {
        // copies already requested still land: wait for them (bounded) before the block exits
        const uint32_t first = it > (uint32_t)S ? it - S : 0;
        for (uint32_t j = first; j < it; ++j) mbar_drain(LBAR(B_FULL + j % S), (j / S) & 1);
      }
    }
  } else if (warp == 1) {
    // ================= MMA issuer =============================================
    if (lane == 0) {
      const uint64_t desc0 = smem_desc_k128(sm_base);
      uint32_t it = 0;
      bool ok = !*abort_flag;
      for (int box = 0; box < nb && ok; ++box) {
        const int buf = box % n_bufs;
        const int row0 = r0 + box * p.n_box;
        const uint32_t idesc = instr_desc((r1 - row0 <= p.tail_rows) ? p.tail_rows : p.n_box);
        if (box >= n_bufs) ok = mbar_wait(LBAR(B_ACCEMPTY + buf), ((box / n_bufs) - 1) & 1, abort_flag, p.err, 2);
        if (!ok) break;
        tc_fence_after();
        for (int kb0 = 0; kb0 < KB; kb0 += kbs, ++it) {
          const int s = it % S;
          const int nk = min(kbs, KB - kb0);
          ok = mbar_wait(LBAR(B_FULL + s), (it / S) & 1, abort_flag, p.err, 3);
          if (!ok) break;
          tc_fence_after();
          const uint32_t st_off = (uint32_t)s * L.stage_bytes;
          for (int j = 0; j < nk; ++j) {
            const uint64_t wd = desc0 + (uint64_t)((st_off + L.b_in_stage + (uint32_t)j * L.b_bytes) >> 4);
            for (int mt = 0; mt < p.n_mt; ++mt) {
              // block rows 128*mt .. of the hidden tile (8-row groups are contiguous: 16 KB further on)
              const uint64_t hd = desc0 + (uint64_t)((st_off + (uint32_t)j * L.a_bytes + (uint32_t)mt * 16384u) >> 4);
              const uint32_t acc = tmem + (uint32_t)((buf * p.n_mt + mt) * LM_MAX_BOX);
#pragma unroll
              for (int kk = 0; kk < LM_KB / 16; ++kk)      // 32 bytes per 16 elements inside the swizzled row
                mma_ss(acc, hd + (uint64_t)(kk * 2), wd + (uint64_t)(kk * 2), idesc, (kb0 | j | kk) ? 1u : 0u);
            }
          }
          tc_commit(LBAR(B_EMPTY + s));
        }
        if (ok) tc_commit(LBAR(B_ACCFULL + buf));
      }
    }
  } else {
    // ================= epilogue ================================================
    const int quarter = warp & 3;                          // TMEM lanes 32*quarter .. +31
    const int ew = warp - 2;
    const int row_a = quarter * 32 + lane;                 // this thread's block rows: row_a and row_a + 128
    // the candidates are an input: fetched now, so that the last block's scan does not wait for them
    for (int t = threadIdx.x - 64; t < p.B * p.k; t += 128) cand_s[t] = p.cand[t];
    float m0 = LM_NEG, s0 = 0.f, m1 = LM_NEG, s1 = 0.f;
    int i0 = 0x7FFFFFFF, i1 = 0x7FFFFFFF;
    const bool sample = p.mode == SPACE_MODE_SAMPLE;
    RowNoisy n0, n1;
    if (sample) { row_noisy_init(n0, p, row_a); row_noisy_init(n1, p, p.n_mt == 2 ? LM_M + row_a : p.n_rows); }
    // a warp whose 32 lanes hold no block row only takes part in the hand-shakes
    const bool warp_a = quarter * 32 < p.n_rows, warp_b = p.n_mt == 2 && LM_M + quarter * 32 < p.n_rows;
    bool ok = true;
    for (int box = 0; box < nb; ++box) {
      const int buf = box % n_bufs;
      ok = ok && mbar_wait(LBAR(B_ACCFULL + buf), (box / n_bufs) & 1, abort_flag, p.err, 4, true);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after();
      const int row0 = r0 + box * p.n_box;
      const int n_valid = min(r1 - row0, (r1 - row0 <= p.tail_rows) ? p.tail_rows : p.n_box);
      const uint32_t acc = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * p.n_mt * LM_MAX_BOX);
      if (warp_a) {
        for (int c0 = 0; c0 < n_valid; c0 += 16) {
          uint32_t v[16];
          tmem_ld16(acc + (uint32_t)c0, v);
          tmem_wait_ld();
          if (sample) fold16_noisy(m0, s0, i0, n0, v, row0 + c0, n_valid - c0, p.c_t, p.key0, p.key1);
          else fold16(m0, s0, i0, v, row0 + c0, n_valid - c0);
        }
      }
      if (warp_b) {
        for (int c0 = 0; c0 < n_valid; c0 += 16) {
          uint32_t v[16];
          tmem_ld16(acc + (uint32_t)(LM_MAX_BOX + c0), v);
          tmem_wait_ld();
          if (sample) fold16_noisy(m1, s1, i1, n1, v, row0 + c0, n_valid - c0, p.c_t, p.key0, p.key1);
          else fold16(m1, s1, i1, v, row0 + c0, n_valid - c0);
        }
      }
      // this accumulator buffer may be overwritten by the products of the next box that uses it
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(LBAR(B_ACCEMPTY + buf));
    }
    // publish this block's statistics of every block row
    if (row_a < p.n_rows) {
      LmPartial out; out.m = m0; out.s = s0; out.idx = i0; out.pad = 0;
      *reinterpret_cast<int4*>(p.part + (size_t)row_a * G + c) = *reinterpret_cast<const int4*>(&out);
      atomicMax(p.keys + row_a, argmax_key(m0, i0));
      if (sample) {
        LmNoisy g; g.gs = n0.gs; g.gz = n0.gz; g.gidx = n0.gidx; g.pad = 0;
        *reinterpret_cast<int4*>(p.gpart + (size_t)row_a * G + c) = *reinterpret_cast<const int4*>(&g);
        if ((unsigned)(n0.cand_tok - r0) < (unsigned)(r1 - r0)) p.zc[row_a] = n0.zc;   // this block owns the candidate's token
      }
    }
    if (p.n_mt == 2 && LM_M + row_a < p.n_rows) {
      LmPartial out; out.m = m1; out.s = s1; out.idx = i1; out.pad = 0;
      *reinterpret_cast<int4*>(p.part + (size_t)(LM_M + row_a) * G + c) = *reinterpret_cast<const int4*>(&out);
      atomicMax(p.keys + LM_M + row_a, argmax_key(m1, i1));
      if (sample) {
        LmNoisy g; g.gs = n1.gs; g.gz = n1.gz; g.gidx = n1.gidx; g.pad = 0;
        *reinterpret_cast<int4*>(p.gpart + (size_t)(LM_M + row_a) * G + c) = *reinterpret_cast<const int4*>(&g);
        if ((unsigned)(n1.cand_tok - r0) < (unsigned)(r1 - r0)) p.zc[LM_M + row_a] = n1.zc;
      }
    }
    __threadfence();
    epi_sync();
    const int et = threadIdx.x - 64;                       // 0..127
    if (et == 0) {
      const int prev = atomicAdd(p.counter, 1);
      const int last = prev == G - 1;
      if (last) *p.counter = 0;                            // ready for the next launch
      *last_flag = last;
    }
    epi_sync();
    if (*last_flag) {
      __threadfence();
      // ---- last thread block.  Every row's (maximum, arg-max) is already combined in its key;
      // only the k mask rows of group i* of every sequence need their sums, so only those rows'
      // per-range partials are read, all of them at once over the 128 threads.
      const int k1 = p.k + 1;
      float* row_m = row_s;                                // [n_rows] maxima (row_s is reused: sums come later)
      int* istar = reinterpret_cast<int*>(smem_raw);       // [B] (the pipeline stages are idle now)
      float* terms = reinterpret_cast<float*>(smem_raw) + LM_MAX_N;   // [B * k][G] scaled sums of the ranges
      for (int r = et; r < p.n_rows; r += 128) {
        const unsigned long long key = atomicExch(p.keys + r, 0ull);      // read, and ready for the next launch
        float m; int idx;
        argmax_unkey(key, m, idx);
        row_m[r] = m; row_i[r] = idx;
        if (p.row_max) p.row_max[r] = m;
        if (p.row_argmax) p.row_argmax[r] = idx;
      }
      epi_sync();
      if (sample) {
        // ---- sampling mode (Algorithm 1 with r <= Q/P_c; see verify.cu for the same steps on
        // stored logits).  tsum: sums of exp2((z - max) c) of the rows named by row_of(b, j),
        // j = 0..k-1, combined from the ranges' partials in a fixed order.
        const float cT = p.c_t;
        float* tsum = reinterpret_cast<float*>(smem_raw) + LM_MAX_N;        // [B * k]
        float* terms2 = tsum + LM_MAX_N;                                    // [B * k][G]
        const bool literal = p.resample == SPACE_RESAMPLE_PAPER_LITERAL;
        auto sum_rows = [&](bool mask_rows) {
          const int total = p.B * p.k * G;
          for (int i0 = et; i0 < total; i0 += 128 * 8) {
            int4 v[8]; float mx[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const int at = i0 + u * 128;
              v[u] = make_int4(0, 0, 0, 0); mx[u] = 0.f;
              if (at < total) {
                const int g = at % G, bj = at / G;
                const int b = bj / p.k, jj = bj - b * p.k;
                const int row = b * p.n_q + (mask_rows ? istar[b] * k1 + jj + 1 : jj * k1);
                mx[u] = row_m[row];
                v[u] = __ldcg(reinterpret_cast<const int4*>(p.part + (size_t)row * G + g));
              }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const int at = i0 + u * 128;
              if (at < total) terms2[at] = __int_as_float(v[u].y) * fast_exp2((__int_as_float(v[u].x) - mx[u]) * cT);
            }
          }
          epi_sync();
          for (int bj = ew; bj < p.B * p.k; bj += 4) {
            float sv = 0.f;
            for (int g = lane; g < G; g += 32) sv += terms2[bj * G + g];
            sv = warp_sum(sv);
            if (lane == 0) tsum[bj] = sv;
          }
          epi_sync();
        };
        // best noisy score of a row over the ranges: larger score, then lower token; every lane gets it
        auto best_noisy = [&](int row, float& gz_out) -> int {
          float gs = -CUDART_INF_F, gz = 0.f; int gi = 0x7FFFFFFF;
          for (int g = lane; g < G; g += 32) {
            const int4 v = __ldcg(reinterpret_cast<const int4*>(p.gpart + (size_t)row * G + g));
            const float s2 = __int_as_float(v.x);
            if (s2 > gs || (s2 == gs && v.z < gi)) { gs = s2; gz = __int_as_float(v.y); gi = v.z; }
          }
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) {
            const float os = __shfl_xor_sync(0xFFFFFFFFu, gs, off);
            const float oz = __shfl_xor_sync(0xFFFFFFFFu, gz, off);
            const int oi = __shfl_xor_sync(0xFFFFFFFFu, gi, off);
            if (os > gs || (os == gs && oi < gi)) { gs = os; gz = oz; gi = oi; }
          }
          gz_out = gz;
          return gi;
        };
        sum_rows(false);                                   // target rows t = 0..k-1 of every sequence
        for (int b = ew; b < p.B; b += 4) {
          const int* ri = row_i + b * p.n_q;
          const int t = lane;
          const int cv = (t < p.k) ? cand_s[b * p.k + t] : -1;
          const bool in_range = cv >= 0 && cv < p.V;
          const unsigned bad = __ballot_sync(0xFFFFFFFFu, t < p.k && !in_range);
          bool okc = false;
          const uint32_t seq = p.seq_id ? p.seq_id[b] : p.seq_base + (uint32_t)b;
          const int Lb = p.kv_len ? p.kv_len[b] : 0;
          if (t < p.k && in_range) {
            const int row = b * p.n_q + t * k1;
            const float zc = __ldcg(p.zc + row);
            const float q = fast_exp2((zc - row_m[row]) * cT) / tsum[b * p.k + t];
            const Philox4 w = philox4x32_10(0u, PURPOSE_ACCEPT, seq, (uint32_t)(Lb + t + 1), p.key0, p.key1);
            const float pc = p.cand_prob[b * p.k + t];
            okc = pc > 0.f && uniform_open(w.x) * pc <= q;  // r <= Q/P_c  <=>  r P_c <= Q
          }
          const unsigned acc_mask = __ballot_sync(0xFFFFFFFFu, okc);
          const int i_star = __ffs(~acc_mask) - 1;          // first candidate that is not accepted (k when all are)
          float gz_unused;
          const int bonus = best_noisy(b * p.n_q + i_star * k1, gz_unused);   // a: the draw of the case i* (row i*)
          const int j = lane;
          const int c_j = __shfl_sync(0xFFFFFFFFu, cv, min(j, p.k - 1));
          const int tok = (j < i_star) ? c_j : (j == i_star ? bonus : -1);
          const bool is_eos = p.eos_id >= 0 && j <= i_star && tok == p.eos_id;
          const unsigned eos_mask = __ballot_sync(0xFFFFFFFFu, is_eos && j < k1);
          const int n_out = eos_mask ? __ffs(eos_mask) - 1 : i_star + 1;
          if (j < k1) p.out_tokens[b * k1 + j] = (j < n_out) ? tok : -1;
          if (j < p.k && !literal) {                        // point-mass drafts: arg-max of mask row (i*, j+1), P_c = 1
            p.next_cand[b * p.k + j] = ri[i_star * k1 + j + 1];
            p.next_cand_prob[b * p.k + j] = 1.f;
          }
          if (j == 0) {
            istar[b] = i_star;
            p.n_accept[b] = i_star;
            p.n_out[b] = n_out;
            p.finished[b] = (uint8_t)(eos_mask != 0);
            if (p.status && bad) atomicOr(p.status + b, SPACE_ST_BAD_CANDIDATE);
          }
        }
        epi_sync();
        if (literal) {
          // candidates sampled from the mask rows of group i*, with their probabilities
          sum_rows(true);
          for (int bj = ew; bj < p.B * p.k; bj += 4) {
            const int b = bj / p.k, jj = bj - b * p.k;
            const int row = b * p.n_q + istar[b] * k1 + jj + 1;
            float gz;
            const int tok = best_noisy(row, gz);
            if (lane == 0) {
              p.next_cand[bj] = tok;
              p.next_cand_prob[bj] = fast_exp2((gz - row_m[row]) * cT) / tsum[bj];
            }
          }
        }
      } else {
      // acceptance scan and emitted tokens: one warp per sequence
      for (int b = ew; b < p.B; b += 4) {
        const int* ri = row_i + b * p.n_q;
        const int cv = (lane < p.k) ? cand_s[b * p.k + lane] : -1;
        const bool in_range = cv >= 0 && cv < p.V;
        const unsigned bad = __ballot_sync(0xFFFFFFFFu, lane < p.k && !in_range);
        const bool match = lane < p.k && in_range && cv == ri[lane * k1];
        const unsigned acc_mask = __ballot_sync(0xFFFFFFFFu, match);
        const int i_star = __ffs(~acc_mask) - 1;            // first candidate that does not match (k when all do)
        const int j = lane;
        const int c_j = __shfl_sync(0xFFFFFFFFu, cv, min(j, p.k - 1));
        const int tok = (j < i_star) ? c_j : (j == i_star ? ri[i_star * k1] : -1);
        const bool is_eos = p.eos_id >= 0 && j <= i_star && tok == p.eos_id;
        const unsigned eos_mask = __ballot_sync(0xFFFFFFFFu, is_eos && j < k1);
        const int n_out = eos_mask ? __ffs(eos_mask) - 1 : i_star + 1;
        if (j < k1) p.out_tokens[b * k1 + j] = (j < n_out) ? tok : -1;
        if (j < p.k) p.next_cand[b * p.k + j] = ri[i_star * k1 + j + 1];  // mask row (i*, j+1)
        if (j == 0) {
          istar[b] = i_star;
          p.n_accept[b] = i_star;
          p.n_out[b] = n_out;
          p.finished[b] = (uint8_t)(eos_mask != 0);
          if (p.status && bad) atomicOr(p.status + b, SPACE_ST_BAD_CANDIDATE);
        }
      }
      epi_sync();
      // sums of the mask rows of group i*: (sequence, mask row, range) triples spread over the threads
      const int total = p.B * p.k * G;
      for (int i0 = et; i0 < total; i0 += 128 * 8) {
        int4 v[8]; float mx[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int at = i0 + u * 128;
          v[u] = make_int4(0, 0, 0, 0); mx[u] = 0.f;
          if (at < total) {
            const int g = at % G, bj = at / G;
            const int b = bj / p.k, jj = bj - b * p.k;
            const int row = b * p.n_q + istar[b] * k1 + jj + 1;
            mx[u] = row_m[row];
            v[u] = __ldcg(reinterpret_cast<const int4*>(p.part + (size_t)row * G + g));
          }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int at = i0 + u * 128;
          if (at < total) terms[at] = __int_as_float(v[u].y) * fast_exp2((__int_as_float(v[u].x) - mx[u]) * LOG2E);
        }
      }
      epi_sync();
      // fixed summation order: the result does not depend on which block came last or on timing
      for (int bj = ew; bj < p.B * p.k; bj += 4) {
        float sv = 0.f;
        for (int g = lane; g < G; g += 32) sv += terms[bj * G + g];
        sv = warp_sum(sv);
        if (lane == 0) p.next_cand_prob[bj] = 1.f / sv;    // softmax at T = 1 of its own maximum
      }
      }
    }
  }
#undef LBAR
  // ---- exit: every role is done (or has given up); free TMEM
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (*abort_flag && threadIdx.x == 0 && p.status) atomicOr(p.status, SPACE_ST_TIMEOUT);
  if (warp == 1)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);
EncodeTiledFn lm_get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = (EncodeTiledFn)ptr;
  }
  return fn;
}
// [rows, D] bf16 matrix with `ld` elements between rows, boxes of box_rows x 64
int lm_make_map(CUtensorMap* tm, const void* base, int64_t rows, int64_t D, int64_t ld, int box_rows) {
  EncodeTiledFn enc = lm_get_encode();
  if (!enc) return SPACE_E_CUDA;
  const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)rows, 1, 1};
  const cuuint64_t strides[3] = {(cuuint64_t)ld * 2, (cuuint64_t)ld * 2 * (cuuint64_t)rows, (cuuint64_t)ld * 2 * (cuuint64_t)rows};
  const cuuint32_t box[4] = {(cuuint32_t)LM_KB, (cuuint32_t)box_rows, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  const CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B,      // measured against 128 B, 64 B, none: 0.4 us better
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SPACE_OK : SPACE_E_CUDA;
}

}  // namespace

size_t lmhead_partial_bytes(int sm_count) {
  return (size_t)LM_MAX_N * sm_count * (sizeof(LmPartial) + sizeof(LmNoisy));
}

namespace {

// One launch: the sequences of `a` (at most LM_MAX_N block rows); seq_base = index of the first
// of them in the caller's batch.
int launch_group(space_ctx* ctx, const space_lmhead_args* a, uint32_t seq_base, cudaStream_t st) {
  LmParams p;
  memset(&p, 0, sizeof(p));
  p.B = a->batch; p.k = a->k; p.V = a->vocab; p.D = a->hidden_dim;
  p.n_q = (a->k + 1) * (a->k + 1);
  p.n_rows = p.B * p.n_q;
  p.n_pad = (p.n_rows + 15) / 16 * 16;
  if (p.n_pad > LM_MAX_N) return SPACE_E_UNSUPPORTED;
  p.n_mt = p.n_pad > LM_M ? 2 : 1;
  int grid = ctx->sm_count;
  const int max_useful = (a->vocab + 31) / 32;             // at least 32 tokens per thread block
  if (grid > max_useful) grid = max_useful;
  if (grid < 1) grid = 1;
  const int max_len = (a->vocab + grid - 1) / grid + 15;   // the longest vocabulary range (boundaries are multiples of 16)
  p.n_box = max_len >= LM_MAX_BOX ? LM_MAX_BOX : (max_len + 15) / 16 * 16;
  p.tail_rows = (((max_len - 1) % p.n_box) + 1 + 15) / 16 * 16;
  // Slices per stage and stages: two slices when that leaves at least three stages (measured 1..4
  // slices on V = 32000, D = 4096: within 3 %), else one; as many stages as fit, at most LM_MAX_STAGES.
  const size_t budget = 220 * 1024;
  int stages = 0;
  for (p.kbs = 2; p.kbs >= 1; --p.kbs) {
    stages = LM_MAX_STAGES;
    while (stages > 1 && LmSmem(p.n_pad, p.n_box, stages, p.kbs).total + 1024 > budget) --stages;
    if (stages >= (p.kbs == 2 ? 3 : 2)) break;
  }
  if (stages < 2) return SPACE_E_UNSUPPORTED;
  p.stages = stages;
  const LmSmem L(p.n_pad, p.n_box, stages, p.kbs);
  if (L.total + 1024 > 227 * 1024) return SPACE_E_UNSUPPORTED;
  p.eos_id = a->eos_id;
  p.mode = a->mode; p.resample = a->resample;
  p.c_t = LOG2E / (a->mode == SPACE_MODE_SAMPLE ? a->temperature : 1.0f);
  p.key0 = (uint32_t)(a->seed & 0xFFFFFFFFull); p.key1 = (uint32_t)(a->seed >> 32);
  p.seq_base = seq_base;
  p.cand_prob = a->cand_prob; p.seq_id = a->seq_id; p.kv_len = a->kv_len;
  p.gpart = reinterpret_cast<LmNoisy*>(ctx->lm_part + (size_t)LM_MAX_N * ctx->sm_count * sizeof(LmPartial));
  p.zc = reinterpret_cast<float*>(reinterpret_cast<char*>(ctx->lm_counter) + 256 + LM_MAX_N * sizeof(unsigned long long));
  p.cand = a->cand;
  p.n_accept = a->n_accept; p.out_tokens = a->out_tokens; p.n_out = a->n_out; p.next_cand = a->next_cand;
  p.next_cand_prob = a->next_cand_prob; p.finished = a->finished; p.status = a->status;
  p.row_max = a->row_max; p.row_argmax = a->row_argmax;
  p.part = reinterpret_cast<LmPartial*>(ctx->lm_part);
  p.counter = ctx->lm_counter;
  p.keys = reinterpret_cast<unsigned long long*>(ctx->lm_counter + 64);
  p.err = ctx->lm_counter + 1;
  int rc = lm_make_map(&p.tm_w, a->weight, a->vocab, a->hidden_dim, a->weight_row_stride, p.n_box);
  if (rc == SPACE_OK) rc = lm_make_map(&p.tm_wt, a->weight, a->vocab, a->hidden_dim, a->weight_row_stride, p.tail_rows);
  if (rc == SPACE_OK) rc = lm_make_map(&p.tm_h, a->hidden, p.n_rows, a->hidden_dim, a->hidden_row_stride, p.n_pad);
  if (rc != SPACE_OK) return rc;
  const size_t sm = L.total + 1024;
  cudaFuncSetAttribute(lmhead_verify_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
  {
    ProfScope ps(ctx, SPACE_K_LMHEAD, st);
    launch_pdl(lmhead_verify_kernel, dim3(grid), dim3(LM_THREADS), sm, st, p);
  }
  ctx->launches += 1;
  return cuda_ok(cudaGetLastError());
}

}  // namespace

// A batch of more block rows than one launch covers goes group of sequences by group of
// sequences: every group streams the output embedding once and is complete in itself (the
// results are per sequence).  The launches follow one another on the stream and share the scratch.
int launch_lmhead_verify(space_ctx* ctx, const space_lmhead_args* a, cudaStream_t st) {
  const int n_q = (a->k + 1) * (a->k + 1), k1 = a->k + 1;
  const int per_group = LM_MAX_N / n_q;
  if (per_group < 1) return SPACE_E_UNSUPPORTED;
  for (int b0 = 0; b0 < a->batch; b0 += per_group) {
    space_lmhead_args g = *a;
    g.batch = a->batch - b0 < per_group ? a->batch - b0 : per_group;
    g.hidden = static_cast<const __nv_bfloat16*>(a->hidden) + (int64_t)b0 * n_q * a->hidden_row_stride;
    g.cand = a->cand + (int64_t)b0 * a->k;
    if (a->cand_prob) g.cand_prob = a->cand_prob + (int64_t)b0 * a->k;
    if (a->seq_id) g.seq_id = a->seq_id + b0;
    if (a->kv_len) g.kv_len = a->kv_len + b0;
    g.n_accept = a->n_accept + b0; g.out_tokens = a->out_tokens + (int64_t)b0 * k1; g.n_out = a->n_out + b0;
    g.next_cand = a->next_cand + (int64_t)b0 * a->k; g.next_cand_prob = a->next_cand_prob + (int64_t)b0 * a->k;
    g.finished = a->finished + b0;
    if (a->status) g.status = a->status + b0;
    if (a->row_max) g.row_max = a->row_max + (int64_t)b0 * n_q;
    if (a->row_argmax) g.row_argmax = a->row_argmax + (int64_t)b0 * n_q;
    const int rc = launch_group(ctx, &g, (uint32_t)b0, st);
    if (rc != SPACE_OK) return rc;
  }
  return SPACE_OK;
}
