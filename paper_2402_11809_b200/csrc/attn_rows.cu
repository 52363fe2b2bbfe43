// Tensor-core attention of the block rows over cache + block (Eq. 5) for sm_100a,
// row orientation: used when the query block of one kv head has more than 64
// rows (block rows times GQA group), where a full 128-row MMA tile is well
// filled.  Narrower blocks go to the transposed kernel of attn_tc.cu, which
// this file mirrors in structure (flat tile partition, split partials, merge).
//
// Here the query rows are the MMA M extent and the 128 keys of a tile the N
// extent: S = Q K^T (128 x 128) into one of two TMEM buffers, P overwrites S in
// TMEM as two bf16 terms, O += (P_hi + P_lo) V with P read back from TMEM.
// Inside a block (12 warps): warps 0 and 2 stream K and V tiles with TMA, warp
// 3 loads the query rows, warp 1 issues tcgen05.mma, warps 4-11 are two threads
// per query row (64 keys of the tile each) with a running row maximum and lazy
// rescaling of O.  Every wait is bounded; an expired wait sets SPACE_ST_TIMEOUT
// and the block drains and exits.
#include "common.cuh"
#include "tc_common.cuh"
#include <cuda.h>
#include <math_constants.h>

namespace {

constexpr int TILE_N = 128;            // keys per tile
constexpr int ROWS = 128;              // MMA M
constexpr int THREADS = 384;            // K (+Q), S-issuer, V, O-issuer warps + 8 softmax warps
constexpr uint64_t WAIT_NS = 1000000000ull;   // one second per wait
constexpr float RESCALE_THRESHOLD = 8.f;
// Starting a share (query load, pipeline refill, epilogue) costs about as much as
// this many tiles; the flat list carries that many extra entries per (sequence, head).
constexpr int SHARE_COST = 4;

struct AttnParams {
  CUtensorMap tm_q, tm_k, tm_v;
  int B, n_q, H_q, H_kv, G;
  int n_mblocks, rows_per_mb;          // query-row blocks per kv head; block rows i per block
  int n_groups;                        // thread-block groups (grid = n_groups * n_mblocks)
  int out_dtype;
  int64_t s_cap;                       // rows a sequence may hold (paged: pages_per_seq * SPACE_PAGE_SIZE)
  // Paged cache (page_table != nullptr): tm_k / tm_v describe a pool [n_pages][H_kv][TILE_N][d] and tile t
  // of sequence b is the whole page page_table[b * pages_per_seq + t]; no tile is shifted back, the
  // rows of the last page past the last key are masked (S) and cleared in shared memory (V).
  const int32_t* page_table; int pages_per_seq, n_pages;
  float scale_log2;                    // scale * log2(e)
  const int32_t* kv_len;
  void* out; float* lse; int32_t* status;
  float* part;                         // [slots][ROWS*(DH+2)]
  int* err;                            // one word: first timeout site
  int2* desc;                          // [B*H_kv*n_mblocks] {first group, number of groups} of each cut
  int* owner;                          // [grid] (sequence, kv head) whose last piece this thread block computed, or -1
  int merge_by_owner;                  // the merge grid is indexed by attention thread block, not by (sequence, head)
  uint64_t mask[SPACE_MAX_ROWS];
};

struct Seg { int b, h, t0, t1, T, L; };

// Page of tile t of sequence b (paged cache).  An entry outside the pool is flagged and answered
// with a page past the pool's end: the TMA load then fills the tile with zeros.
__device__ __forceinline__ int page_of(const AttnParams& p, int b, int t) {
  const int pg = t < p.pages_per_seq ? p.page_table[(int64_t)b * p.pages_per_seq + t] : -1;
  if (pg >= 0 && pg < p.n_pages) return pg;
  if (p.status) atomicOr(p.status + b, SPACE_ST_BAD_PAGE);
  return p.n_pages;
}

// PTX helpers: tc_common.cuh.  Every wait of this kernel is bounded by WAIT_NS.
using namespace tc;
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* err, int site) {
  return mbar_wait_bounded(bar, parity, abort_flag, err, site, WAIT_NS, 0);
}
__device__ __forceinline__ void mbar_drain(uint32_t bar, uint32_t parity) { mbar_drain_bounded(bar, parity, WAIT_NS); }
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
// Instruction descriptor: bf16 x bf16 -> f32, M = 128.
__host__ __device__ constexpr uint32_t instr_desc(int n, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(ROWS >> 4) << 24);
}

// ------------------------------------------------------------ work partition
// Flat tile index space: sequence-major, then kv head, then tile.  Group g of
// n_groups owns flat tiles [W*g/n_groups, W*(g+1)/n_groups).
// floor(a * b / c) for a*b that may need 64 bits; 32-bit division when it fits
__device__ __forceinline__ long long muldiv(long long a, long long b, long long c) {
  const unsigned long long prod = (unsigned long long)a * (unsigned long long)b;
  if ((prod >> 32) == 0) return (long long)((unsigned)prod / (unsigned)c);
  return (long long)(prod / (unsigned long long)c);
}

struct Partition {
  const int* seq_len;    // [B]   verified length, or -1 for a sequence that does not fit
  const int* prefix;     // [B+1] flat offset of sequence b
  int B, H_kv, n_q;
  long long cur, end;
  int b;
  // Only min(n_groups, W) groups take part, so every taking-part group owns at
  // least one tile and the groups of one (sequence, head) are consecutive.
  __device__ void init(const int* sl, const int* pf, int B_, int H, int nq, int group, int n_groups) {
    seq_len = sl; prefix = pf; B = B_; H_kv = H; n_q = nq; b = 0;
    const long long W = pf[B_];
    const long long NG = W < n_groups ? W : n_groups;
    if (group >= NG) { cur = end = 0; return; }
    cur = muldiv(W, group, NG);
    end = muldiv(W, group + 1, NG);
  }
  __device__ bool next(Seg& s) {
    // The list holds T + SHARE_COST entries per (sequence, head); the first
    // SHARE_COST stand for the fixed cost of starting a share there, so that
    // equal list shares are shares of about equal time.
    for (;;) {
      if (cur >= end) return false;
      while (prefix[b + 1] <= cur) ++b;
      const int L = seq_len[b];
      const int T = (L + n_q + TILE_N - 1) / TILE_N;
      const int Tv = T + SHARE_COST;
      const int rem = (int)(cur - prefix[b]);
      const int h = rem / Tv, r0 = rem - h * Tv;
      long long n = Tv - r0;
      if (n > end - cur) n = end - cur;
      cur += n;
      const int t0 = max(r0 - SHARE_COST, 0), t1 = max(r0 + (int)n - SHARE_COST, 0);
      if (t1 <= t0) continue;                               // only cost entries here: no tiles
      s.b = b; s.h = h; s.t0 = t0; s.t1 = t1; s.T = T; s.L = L;
      return true;
    }
  }
};

// group that owns flat tile f (largest g with floor(W*g/NG) <= f)
__device__ __forceinline__ int group_of(long long f, long long W, long long NG) {
  const unsigned long long num = (unsigned long long)(f + 1) * (unsigned long long)NG - 1ull;
  if ((num >> 32) == 0) return (int)((unsigned)num / (unsigned)W);
  return (int)(num / (unsigned long long)W);
}

template <int DH>
struct Smem {
  static constexpr int HALVES = DH / 64;
  static constexpr int TILE_BYTES = TILE_N * DH * 2;         // one K or V tile
  static constexpr int Q_BYTES = ROWS * DH * 2;
  static constexpr int K_STAGES = (DH == 128) ? 2 : 3;
  static constexpr int V_STAGES = (DH == 128) ? 2 : 4;
  static constexpr int Q_OFF = 0;
  static constexpr int K_OFF = Q_BYTES;
  static constexpr int V_OFF = K_OFF + K_STAGES * TILE_BYTES;
  static constexpr int BAR_OFF = V_OFF + V_STAGES * TILE_BYTES;
  static constexpr int S_BUFS = 3;                           // S / P buffers in TMEM (3 x 128 columns, O at 384)
  // q_full, q_empty, k_full[], k_empty[], v_full[], v_empty[], s_full[3], p_ready[3], pv_done[3], drain
  static constexpr int N_BARS = 2 + 2 * K_STAGES + 2 * V_STAGES + 3 * S_BUFS + 1;
  static constexpr int MISC_OFF = BAR_OFF + (N_BARS * 8 + 15) / 16 * 16;   // tmem base, abort flag
  static constexpr int XMAX_OFF = MISC_OFF + 32;             // [2 parities][2 halves][ROWS] float
  static constexpr int XSUM_OFF = XMAX_OFF + 2 * 2 * ROWS * 4;   // [2 halves][ROWS] float
  static constexpr int EPI_PITCH = 36;                       // floats per staged row: 32 columns + 4 (16-byte aligned, conflict-free)
  static constexpr int EPI_OFF = XSUM_OFF + 2 * ROWS * 4;    // [8 warps][32 rows][EPI_PITCH] float: epilogue transpose
  static constexpr int TABLE_OFF = EPI_OFF + 8 * 32 * EPI_PITCH * 4;   // seq_len[max_batch], prefix[max_batch+1]
};


// The two softmax warps that share a TMEM lane quarter meet here (ids 1..4).
__device__ __forceinline__ void pair_sync(int quarter) {
  asm volatile("bar.sync %0, 64;" ::"r"(quarter + 1) : "memory");
}

// Warp roles
constexpr int WARP_K = 0, WARP_MMA = 1, WARP_V = 2, WARP_PV = 3, WARP_SOFTMAX0 = 4;

template <int DH>
__global__ void __launch_bounds__(THREADS, 1) attn_rows_kernel(const __grid_constant__ AttnParams p,
                                                             int max_batch) {
  using S = Smem<DH>;
  extern __shared__ __align__(1024) unsigned char sm[];
  const uint32_t sm_base = smem_u32(sm);
  const uint32_t bar0 = sm_base + S::BAR_OFF;
  auto BAR = [&](int i) { return bar0 + 8u * i; };
  constexpr int B_QFULL = 0, B_QEMPTY = 1, B_KFULL = 2, B_KEMPTY = B_KFULL + S::K_STAGES,
                B_VFULL = B_KEMPTY + S::K_STAGES, B_VEMPTY = B_VFULL + S::V_STAGES,
                B_SFULL = B_VEMPTY + S::V_STAGES, B_PREADY = B_SFULL + S::S_BUFS,
                B_PVDONE = B_SFULL + 2 * S::S_BUFS, B_DRAIN = B_SFULL + 3 * S::S_BUFS;
  constexpr uint32_t NS = S::S_BUFS;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + S::MISC_OFF);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + S::MISC_OFF + 4);
  float* xmax = reinterpret_cast<float*>(sm + S::XMAX_OFF);
  float* xsum = reinterpret_cast<float*>(sm + S::XSUM_OFF);
  int* seq_len = reinterpret_cast<int*>(sm + S::TABLE_OFF);
  int* prefix = seq_len + max_batch;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int group = blockIdx.x / p.n_mblocks, mb = blockIdx.x % p.n_mblocks;
  const int i0 = mb * p.rows_per_mb;                       // first block row of this query-row block
  // MMA rows that carry a real (block row, head) pair are 0 .. m_valid-1
  const int m_valid = min(p.rows_per_mb, p.n_q - i0) * p.G;
  const int n_quarters = (m_valid + 31) >> 5;              // TMEM lane quarters with live rows
  const int n_soft = 64 * n_quarters;                      // softmax threads that take part

  // ---- set-up ------------------------------------------------------------
  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    *abort_flag = (sm_base & 1023u) ? 1 : 0;               // swizzled tiles need a 1024-byte aligned base
    mbar_init(BAR(B_QFULL), 1);
    mbar_init(BAR(B_QEMPTY), 1);
    for (int s = 0; s < S::K_STAGES; ++s) { mbar_init(BAR(B_KFULL + s), 1); mbar_init(BAR(B_KEMPTY + s), 1); }
    for (int s = 0; s < S::V_STAGES; ++s) { mbar_init(BAR(B_VFULL + s), 1); mbar_init(BAR(B_VEMPTY + s), 1); }
    for (int i = 0; i < S::S_BUFS; ++i) {
      mbar_init(BAR(B_SFULL + i), 1);
      mbar_init(BAR(B_PREADY + i), n_soft);
      mbar_init(BAR(B_PVDONE + i), 1);
    }
    mbar_init(BAR(B_DRAIN), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  pdl_wait();                                              // global memory from here on
  if (warp == WARP_SOFTMAX0) {
    // per-sequence tile counts and their running sum, 32 sequences per round
    int carry = 0;
    for (int b0 = 0; b0 < p.B; b0 += 32) {
      const int b = b0 + lane;
      int L = -1, tiles = 0;
      if (b < p.B) {
        L = p.kv_len[b];
        const bool ok = L >= 0 && (int64_t)L + p.n_q <= p.s_cap;
        if (!ok && blockIdx.x == 0 && p.status) atomicOr(p.status + b, SPACE_ST_CAPACITY);
        if (!ok) L = -1;
        tiles = ok ? ((L + p.n_q + TILE_N - 1) / TILE_N + SHARE_COST) * p.H_kv : 0;
      }
      int incl = tiles;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += v;
      }
      if (b < p.B) { seq_len[b] = L; prefix[b] = carry + incl - tiles; }
      carry += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
    if (lane == 0) prefix[p.B] = carry;
  }
  if (warp == WARP_MMA) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (warp == WARP_K && lane == 0)
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&p.tm_k) : "memory");
  if (warp == WARP_V && lane == 0)
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&p.tm_v) : "memory");
  if (warp == WARP_MMA && lane == 0)
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&p.tm_q) : "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t TM_S0 = tmem, TM_O = tmem + S::S_BUFS * TILE_N;   // S buffers at columns 0, 128, 256; O at 384

  Partition part;
  part.init(seq_len, prefix, p.B, p.H_kv, p.n_q, group, p.n_groups);
  Seg sg;
  const bool dead = *abort_flag != 0;

  if (dead) {
    // nothing was issued; fall through to the teardown
  } else if (warp == WARP_K || warp == WARP_V) {
    // ================= K / V producers ====================================
    if (lane == 0) {
      const bool is_k = warp == WARP_K;
      const int n_st = is_k ? S::K_STAGES : S::V_STAGES;
      const int b_full = is_k ? B_KFULL : B_VFULL, b_empty = is_k ? B_KEMPTY : B_VEMPTY;
      const uint32_t ring = sm_base + (is_k ? S::K_OFF : S::V_OFF);
      const CUtensorMap* tm = is_k ? &p.tm_k : &p.tm_v;
      uint32_t gt = 0, seg = 0;
      bool ok = true;
      while (ok && part.next(sg)) {
        const int n_keys = sg.L + p.n_q;
        if (is_k) {
          // the K producer also loads this share's query rows, once the last S
          // product of the share before has read the buffer
          if (seg > 0) ok = mbar_wait(BAR(B_QEMPTY), (seg - 1) & 1, abort_flag, p.err, 3);
          if (!ok) break;
          mbar_expect_tx(BAR(B_QFULL), S::Q_BYTES);
#pragma unroll
          for (int hf = 0; hf < S::HALVES; ++hf)
            tma_load_4d(sm_base + S::Q_OFF + hf * (ROWS * 128), &p.tm_q, BAR(B_QFULL), hf * 64,
                        sg.h * p.G, i0, sg.b);
          ++seg;
        }
        for (int t = sg.t0; t < sg.t1 && ok; ++t, ++gt) {
          const int s = gt % n_st;
          if (gt >= (uint32_t)n_st)
            ok = mbar_wait(BAR(b_empty + s), ((gt / n_st) - 1) & 1, abort_flag, p.err, is_k ? 1 : 2);
          if (!ok) break;
          // the last tile of a sequence is shifted back so that it ends at the
          // last key: rows past the end are never read (they may hold anything)
          // (a paged cache has whole pages for tiles instead; see AttnParams)
          const int kt = p.page_table ? 0 : (((t + 1) * TILE_N <= n_keys) ? t * TILE_N : n_keys - TILE_N);
          const int kb = p.page_table ? page_of(p, sg.b, t) : sg.b;
          const uint32_t dst = ring + s * S::TILE_BYTES;
          mbar_expect_tx(BAR(b_full + s), S::TILE_BYTES);
#pragma unroll
          for (int hf = 0; hf < S::HALVES; ++hf)
            tma_load_4d(dst + hf * (TILE_N * 128), tm, BAR(b_full + s), hf * 64, kt, sg.h, kb);
        }
      }
      // drain: every issued copy must have landed before the block may exit
      const uint32_t first = gt > (uint32_t)n_st ? gt - n_st : 0;
      for (uint32_t g = first; g < gt; ++g) mbar_drain(BAR(b_full + g % n_st), (g / n_st) & 1);
      if (is_k && seg > 0) mbar_drain(BAR(B_QFULL), (seg - 1) & 1);
    }
  } else if (warp == WARP_MMA) {
    // ================= S issuer ============================================
    if (lane == 0) {
      constexpr uint32_t IDESC_QK = instr_desc(TILE_N, 0);
      uint32_t gt = 0, seg = 0;
      bool ok = true;
      while (ok && part.next(sg)) {
        ok = mbar_wait(BAR(B_QFULL), seg & 1, abort_flag, p.err, 6);
        const int n = sg.t1 - sg.t0;
        for (int j = 0; j < n && ok; ++j, ++gt) {
          const int s = gt % S::K_STAGES;
          const uint32_t buf = gt % NS;
          ok = mbar_wait(BAR(B_KFULL + s), (gt / S::K_STAGES) & 1, abort_flag, p.err, 7);
          // S buffer `buf` held the P of tile gt - 3, read by that tile's O product
          if (ok && gt >= NS) ok = mbar_wait(BAR(B_PVDONE + buf), ((gt / NS) - 1) & 1, abort_flag, p.err, 8);
          if (!ok) break;
          tc_fence_after();
          const uint32_t qsm = sm_base + S::Q_OFF;
          const uint32_t ksm = sm_base + S::K_OFF + s * S::TILE_BYTES;
#pragma unroll
          for (int kk = 0; kk < DH / 16; ++kk) {
            const uint32_t off = (kk >> 2) * (ROWS * 128) + (kk & 3) * 32;   // 64-wide half, then 32 B per 16 elements
            mma_ss(TM_S0 + buf * TILE_N, smem_desc(qsm + off, 16, 1024), smem_desc(ksm + off, 16, 1024),
                   IDESC_QK, kk > 0 ? 1u : 0u);
          }
          tc_commit(BAR(B_SFULL + buf));
          tc_commit(BAR(B_KEMPTY + s));
          if (j == n - 1) tc_commit(BAR(B_QEMPTY));
        }
        ++seg;
      }
    }
  } else if (warp == WARP_PV) {
    // ================= O issuer ============================================
    // A thread of its own: the S products of later tiles need not queue behind
    // the sixteen instructions of an O product or wait for its operands.
    if (lane == 0) {
      constexpr uint32_t IDESC_PV = instr_desc(DH, 1);
      uint32_t g = 0;
      bool ok = true;
      while (ok && part.next(sg)) {
        for (int t = sg.t0; t < sg.t1 && ok; ++t, ++g) {
          // O += (P_hi + P_lo) V; the first product of a share overwrites O
          const int s = g % S::V_STAGES;
          const uint32_t buf = g % NS;
          ok = mbar_wait(BAR(B_VFULL + s), (g / S::V_STAGES) & 1, abort_flag, p.err, 4);
          if (ok) ok = mbar_wait(BAR(B_PREADY + buf), (g / NS) & 1, abort_flag, p.err, 5);
          if (!ok) break;
          tc_fence_after();
          const uint32_t vsm = sm_base + S::V_OFF + s * S::TILE_BYTES;
          const uint32_t ptm = TM_S0 + buf * TILE_N;
#pragma unroll
          for (int part_i = 0; part_i < 2; ++part_i) {        // P_hi, then P_lo
#pragma unroll
            for (int kk = 0; kk < TILE_N / 16; ++kk) {
              // V tile is MN-major: 64-wide d blocks TILE_N*128 bytes apart, 8-key groups 1024 bytes apart
              const uint64_t bd = smem_desc(vsm + kk * 2048, TILE_N * 128, 1024);
              mma_ts(TM_O, ptm + part_i * (TILE_N / 2) + kk * 8, bd, IDESC_PV,
                     (t == sg.t0 && kk == 0 && part_i == 0) ? 0u : 1u);
            }
          }
          tc_commit(BAR(B_VEMPTY + s));
          tc_commit(BAR(B_PVDONE + buf));
        }
      }
      // all tensor work done before TMEM is released (every S product was read by
      // the softmax before the O product that follows it was issued)
      tc_commit(BAR(B_DRAIN));
      mbar_drain(BAR(B_DRAIN), 0);
    }
  } else if ((warp & 3) < n_quarters) {
    // ================= softmax / epilogue ==================================
    // Two threads per query row: `half` picks which 64 keys of a tile (and which
    // half of the head dimension in the epilogue) this thread handles.
    const int quarter = warp & 3;                          // TMEM lane quarter this warp may touch
    const int half = (warp - WARP_SOFTMAX0) >> 2;
    const int m = quarter * 32 + lane;                     // MMA row
    const int il = m / p.G, g = m % p.G;
    const int i = i0 + il;                                 // block row
    const bool row_valid = m < m_valid;
    const uint64_t mrow = row_valid ? p.mask[i] : 0ull;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const int sidx = half * (32 * n_quarters) + m;          // index among the n_soft softmax threads
    const float c = p.scale_log2;
    constexpr int HC = TILE_N / 2;                         // keys per thread and tile
    constexpr int OC = DH / 2;                             // output columns per thread
    uint32_t gt = 0;
    // A failed (expired) wait does not leave the loops: every thread keeps the
    // same control flow so that the pair barriers below always match up; once
    // the abort flag is set all later waits return at once and the block drains.
    bool ok = true;
    int own = -1;                                          // item whose last piece of a cut this block holds
    while (part.next(sg)) {
      const int n_keys = sg.L + p.n_q;
      float m_ref = -CUDART_INF_F, l_sum = 0.f;
      for (int t = sg.t0; t < sg.t1; ++t, ++gt) {
        const uint32_t buf = gt % NS;
        ok &= mbar_wait(BAR(B_SFULL + buf), (gt / NS) & 1, abort_flag, p.err, 9);
        tc_fence_after();
        const uint32_t ts = TM_S0 + buf * TILE_N + lane_addr;
        uint32_t sreg[HC];
#pragma unroll
        for (int cc = 0; cc < HC / 32; ++cc) tmem_ld32(ts + half * HC + cc * 32, sreg + cc * 32);
        tmem_wait_ld();
        const int lo = t * TILE_N;
        const int kt = (p.page_table || (t + 1) * TILE_N <= n_keys) ? lo : n_keys - TILE_N;
        const bool masked = (kt + TILE_N > sg.L) || (kt < lo);   // (rows of a page past the last key: no mask bit names them)
        float tmax = -CUDART_INF_F;
        if (masked) {
          // Visibility of this thread's 64 keys as one 64-bit word (bit c: key k0 + c):
          // keys before `lo` belong to the previous tile; cached keys (< L) are seen by
          // every row; block keys by the Eq. 5 mask row of this query row.
          const int k0 = kt + half * HC;
          const int sh = sg.L - k0;                         // first block key sits at bit `sh`
          uint64_t vis;
          if (sh >= 64) vis = ~0ull;
          else if (sh > 0) vis = ((1ull << sh) - 1ull) | (mrow << sh);
          else if (sh > -64) vis = mrow >> (-sh);
          else vis = 0ull;
          const int below = lo - k0;                        // keys k0 .. lo-1 are not this tile's
          if (below >= 64) vis = 0ull;
          else if (below > 0) vis &= ~0ull << below;
          const uint32_t v0 = (uint32_t)vis, v1 = (uint32_t)(vis >> 32);
#pragma unroll
          for (int cidx = 0; cidx < HC; ++cidx) {
            const uint32_t w = cidx < 32 ? v0 : v1;
            const float v = ((w >> (cidx & 31)) & 1u) ? __uint_as_float(sreg[cidx]) : -CUDART_INF_F;
            sreg[cidx] = __float_as_uint(v);
          }
        }
        {
          // four independent running maxima: one chain over 64 values would cost 64 dependent steps
          float t4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
          for (int cidx = 0; cidx < HC; ++cidx) t4[cidx & 3] = fmaxf(t4[cidx & 3], __uint_as_float(sreg[cidx]));
          tmax = fmaxf(fmaxf(t4[0], t4[1]), fmaxf(t4[2], t4[3]));
        }
        // the row maximum needs the other half's keys; the pair barrier also orders
        // both threads' reads of S before either overwrites it with P
        float* xm = xmax + (gt & 1) * (2 * ROWS);
        xm[half * ROWS + m] = tmax;
        pair_sync(quarter);
        tmax = fmaxf(tmax, xm[(half ^ 1) * ROWS + m]);
        tmax *= c;                                         // c > 0
        if (!(tmax > -CUDART_INF_F)) tmax = -CUDART_INF_F; // also catches NaN
        const bool first = (t == sg.t0);
        const bool need = !first && (tmax > m_ref + RESCALE_THRESHOLD);
        if (first) m_ref = tmax;
        if (__any_sync(0xFFFFFFFFu, need)) {
          // lazy rescale of this row's accumulator; PV of the previous tile must be done
          ok &= mbar_wait(BAR(B_PVDONE + (gt - 1) % NS), ((gt - 1) / NS) & 1, abort_flag, p.err, 10);
          tc_fence_after();
          const float m_new = fmaxf(m_ref, tmax);
          const float f = (m_ref > -CUDART_INF_F) ? fast_exp2(m_ref - m_new) : 0.f;
          l_sum *= f;
          m_ref = m_new;
#pragma unroll 1
          for (int cc = 0; cc < OC / 32; ++cc) {
            uint32_t o[32];
            const uint32_t ta = TM_O + lane_addr + half * OC + cc * 32;
            tmem_ld32(ta, o);
            tmem_wait_ld();
#pragma unroll
            for (int x = 0; x < 32; ++x) o[x] = __float_as_uint(__uint_as_float(o[x]) * f);
            tmem_st32(ta, o);
          }
          tmem_wait_st();
        }
        const float m_use = (m_ref > -CUDART_INF_F) ? m_ref : 0.f;
        // P = P_hi + P_lo, two bf16 terms: bf16 alone (8 significant bits) leaves
        // an output error near 1e-2 of the output RMS.  P_hi occupies columns
        // 0..63 of the S buffer, P_lo columns 64..127 (two keys per column).
        uint32_t lreg[HC / 2];
#pragma unroll
        for (int x = 0; x < HC / 2; ++x) {
          const float p0 = fast_exp2(fmaf(__uint_as_float(sreg[2 * x]), c, -m_use));
          const float p1 = fast_exp2(fmaf(__uint_as_float(sreg[2 * x + 1]), c, -m_use));
          l_sum += p0 + p1;
          const __nv_bfloat162 hi = __floats2bfloat162_rn(p0, p1);   // .x (low half) = even key
          const float2 hf = __bfloat1622float2(hi);
          const __nv_bfloat162 lw = __floats2bfloat162_rn(p0 - hf.x, p1 - hf.y);
          sreg[x] = *reinterpret_cast<const uint32_t*>(&hi);
          lreg[x] = *reinterpret_cast<const uint32_t*>(&lw);
        }
        tmem_st32(ts + half * (HC / 2), sreg);
        tmem_st32(ts + TILE_N / 2 + half * (HC / 2), lreg);
        tmem_wait_st();
        if (p.page_table && kt + TILE_N > n_keys) {
          // Paged cache, last tile: the page's rows past the last key may hold anything, and 0 * NaN
          // would reach the output.  Once the V tile has landed the softmax threads clear those rows
          // (128 contiguous bytes per row and 64-wide half of d, whatever the swizzle inside them).
          // The softmax may run up to NS tiles ahead of the O product, the V ring has fewer stages:
          // first make sure that the stage's previous tile has been consumed, so that the wait below
          // looks at the barrier phase of THIS tile and the stores cannot hit the tile before it.
          const uint32_t vs = gt % S::V_STAGES;
          if (gt >= (uint32_t)S::V_STAGES) {
            const uint32_t pg = gt - S::V_STAGES;
            ok &= mbar_wait(BAR(B_PVDONE + pg % NS), (pg / NS) & 1, abort_flag, p.err, 18);
          }
          ok &= mbar_wait(BAR(B_VFULL + vs), (gt / S::V_STAGES) & 1, abort_flag, p.err, 17);
          const int first_bad = n_keys - kt;
          for (int it = first_bad * S::HALVES + sidx; it < TILE_N * S::HALVES; it += n_soft) {
            const int r = it / S::HALVES, hf = it % S::HALVES;
            const uint32_t vrow = sm_base + S::V_OFF + vs * S::TILE_BYTES + hf * (TILE_N * 128) + r * 128;
#pragma unroll
            for (int x = 0; x < 8; ++x)
              asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(vrow + x * 16), "r"(0u) : "memory");
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        tc_fence_before();
        mbar_arrive(BAR(B_PREADY + buf));
      }
      // ---- end of share: final output or partial ---------------------------
      ok &= mbar_wait(BAR(B_PVDONE + (gt - 1) % NS), ((gt - 1) / NS) & 1, abort_flag, p.err, 11);
      tc_fence_after();
      xsum[half * ROWS + m] = l_sum;
      pair_sync(quarter);
      const float l_tot = l_sum + xsum[(half ^ 1) * ROWS + m];
      const bool whole = (sg.t0 == 0 && sg.t1 == sg.T);
      const int hq = sg.h * p.G + g;
      const int item = sg.b * p.H_kv + sg.h;
      float* pslot = p.part + ((size_t)(item + group) * p.n_mblocks + mb) * (ROWS * (DH + 2));
      const float inv = (l_tot > 0.f) ? 1.f / l_tot : 0.f;
      if (sidx == 0 && ok) {
        // how this (sequence, head) was cut: first group and number of groups,
        // read by attn_rows_merge_kernel (every group of the cut writes the same pair)
        int2 d = make_int2(group, 1);
        if (!whole) {
          const long long W = prefix[p.B];
          const long long NG = W < p.n_groups ? W : p.n_groups;
          const long long f0 = (long long)prefix[sg.b] + (long long)sg.h * (sg.T + SHARE_COST) + SHARE_COST;
          d.x = group_of(f0, W, NG);                        // group of the first tile
          d.y = group_of(f0 + sg.T - 1, W, NG) - d.x + 1;
        }
        p.desc[(size_t)item * p.n_mblocks + mb] = d;
        if (sg.t0 > 0 && sg.t1 == sg.T) own = item;        // at most one per block: only its first share can start late
      }
      // O leaves TMEM with one row per lane; written like that, a store instruction
      // would touch 32 different lines.  Each warp turns its 32 x 32 block through
      // shared memory so that eight lanes write 128 contiguous bytes of one row.
      float* stg = reinterpret_cast<float*>(sm + S::EPI_OFF) + (warp - WARP_SOFTMAX0) * (32 * S::EPI_PITCH);
      const int gsh = __ffs(p.G) - 1;                       // G is a power of two
      const float scale_o = whole ? inv : 1.f;
#pragma unroll 1
      for (int cc = 0; cc < OC / 32; ++cc) {
        uint32_t o[32];
        const int col = half * OC + cc * 32;
        tmem_ld32(TM_O + lane_addr + col, o);
        tmem_wait_ld();
#pragma unroll
        for (int x = 0; x < 8; ++x)
          *reinterpret_cast<float4*>(stg + lane * S::EPI_PITCH + 4 * x) =
              make_float4(__uint_as_float(o[4 * x]) * scale_o, __uint_as_float(o[4 * x + 1]) * scale_o,
                          __uint_as_float(o[4 * x + 2]) * scale_o, __uint_as_float(o[4 * x + 3]) * scale_o);
        __syncwarp();
#pragma unroll
        for (int it = 0; it < 8; ++it) {
          const int rl = it * 4 + (lane >> 3), c4 = (lane & 7) * 4;   // row within the warp's block, first of 4 columns
          const int mr = quarter * 32 + rl;
          const float4 v = *reinterpret_cast<const float4*>(stg + rl * S::EPI_PITCH + c4);
          if (mr >= m_valid || !ok) continue;
          if (whole) {
            const int ir = i0 + (mr >> gsh), hr = sg.h * p.G + (mr & (p.G - 1));
            const size_t off = (((size_t)sg.b * p.n_q + ir) * p.H_q + hr) * DH + col + c4;
            if (p.out_dtype == SPACE_DTYPE_F32) {
              *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + off) = v;
            } else {
              const __nv_bfloat162 a0 = __floats2bfloat162_rn(v.x, v.y), a1 = __floats2bfloat162_rn(v.z, v.w);
              *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.out) + off) =
                  make_uint2(*reinterpret_cast<const uint32_t*>(&a0), *reinterpret_cast<const uint32_t*>(&a1));
            }
          } else {
            *reinterpret_cast<float4*>(pslot + (size_t)mr * DH + col + c4) = v;
          }
        }
        __syncwarp();                                       // the block is rewritten by the next chunk
      }
      tc_fence_before();
      if (row_valid && half == 0 && ok) {
        if (whole) {
          if (p.lse)
            p.lse[((size_t)sg.b * p.H_q + hq) * p.n_q + i] = (m_ref + log2f(l_tot)) * 0.6931471805599453f;
        } else {
          pslot[ROWS * DH + m] = m_ref;
          pslot[ROWS * DH + ROWS + m] = l_tot;
        }
      }
    }
    if (sidx == 0) p.owner[blockIdx.x] = own;
  }

  // ---- teardown -----------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == WARP_MMA) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag && p.status) {
    for (int b = 0; b < p.B; ++b) atomicOr(p.status + b, SPACE_ST_TIMEOUT);
  }
}

// Combine the partials of every (sequence, kv head, query-row block) that was
// cut over several groups: one thread per 16 output bytes, all loads of a
// thread independent, running maximum / denominator / accumulator in one pass.
// grid = (B*H_kv*n_mblocks, ceil(rows*DH/4 / 128)), 128 threads.
template <int DH>
__global__ void __launch_bounds__(128) attn_rows_merge_kernel(const AttnParams p) {
  pdl_launch_dependents();
  pdl_wait();
  constexpr int C4 = DH / 4;
  // Large batches: one grid column per attention thread block (each holds the last
  // piece of at most one cut); small ones: one per (sequence, head, row block).
  int item = blockIdx.x / p.n_mblocks;
  const int mb = blockIdx.x % p.n_mblocks;
  if (p.merge_by_owner) {
    item = p.owner[blockIdx.x];
    if (item < 0) return;
  }
  const int b = item / p.H_kv, h = item % p.H_kv;
  // both loads are issued before either is tested: one round trip, not two
  const int L = __ldcg(p.kv_len + b);
  const int2 d = __ldcg(p.desc + (size_t)item * p.n_mblocks + mb);
  if (L < 0 || (int64_t)L + p.n_q > p.s_cap) return;
  const int n = d.y;
  if (n <= 1) return;                                       // written directly by the main kernel
  const int i0 = mb * p.rows_per_mb;
  const int m_valid = min(p.rows_per_mb, p.n_q - i0) * p.G;
  const int idx = blockIdx.y * 128 + threadIdx.x;
  if (idx >= m_valid * C4) return;
  const int r = idx / C4, c4 = idx % C4;
  const size_t slot_floats = (size_t)ROWS * (DH + 2);
  const float* ps = p.part + ((size_t)(item + d.x) * p.n_mblocks + mb) * slot_floats;
  const size_t gstride = (size_t)p.n_mblocks * slot_floats;
  float mx = -CUDART_INF_F, den = 0.f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
  for (int x = 0; x < n; ++x, ps += gstride) {
    const float ms = __ldcg(ps + ROWS * DH + r), ls = __ldcg(ps + ROWS * DH + ROWS + r);
    const float4 ov = __ldcg(reinterpret_cast<const float4*>(ps + (size_t)r * DH) + c4);
    const float mn = fmaxf(mx, ms);
    if (mn > -CUDART_INF_F) {
      const float e0 = fast_exp2(mx - mn), e1 = fast_exp2(ms - mn);
      den = den * e0 + ls * e1;
      acc.x = acc.x * e0 + ov.x * e1; acc.y = acc.y * e0 + ov.y * e1;
      acc.z = acc.z * e0 + ov.z * e1; acc.w = acc.w * e0 + ov.w * e1;
    }
    mx = mn;
  }
  const float rd = 1.f / den;
  const int ri = i0 + r / p.G, hq = h * p.G + r % p.G;
  const size_t off = (((size_t)b * p.n_q + ri) * p.H_q + hq) * DH + c4 * 4;
  if (p.out_dtype == SPACE_DTYPE_F32) {
    *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + off) =
        make_float4(acc.x * rd, acc.y * rd, acc.z * rd, acc.w * rd);
  } else {
    const __nv_bfloat162 a = __floats2bfloat162_rn(acc.x * rd, acc.y * rd);
    const __nv_bfloat162 b2 = __floats2bfloat162_rn(acc.z * rd, acc.w * rd);
    *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.out) + off) =
        make_uint2(*reinterpret_cast<const uint32_t*>(&a), *reinterpret_cast<const uint32_t*>(&b2));
  }
  if (p.lse && c4 == 0)
    p.lse[((size_t)b * p.H_q + hq) * p.n_q + ri] = (mx + log2f(den)) * 0.6931471805599453f;
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
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

int make_map(CUtensorMap* tm, const void* base, const cuuint64_t dims[4], const cuuint64_t strides_bytes[3],
             const cuuint32_t box[4]) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return SPACE_E_CUDA;
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  const CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides_bytes,
                         box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SPACE_OK : SPACE_E_CUDA;
}

void plan(const space_config* cfg, int sm_count, int k, AttnPlanHost* pl) {
  const int G = cfg->n_q_heads / cfg->n_kv_heads;
  const int n_q = (k + 1) * (k + 1);
  const int max_rows = ROWS / G;                            // block rows one MMA tile can hold
  pl->n_mblocks = (n_q + max_rows - 1) / max_rows;
  pl->rows_per_mblock = (n_q + pl->n_mblocks - 1) / pl->n_mblocks;
  int groups = sm_count / pl->n_mblocks;
  if (groups < 1) groups = 1;
  pl->n_ctas = groups * pl->n_mblocks;
}

template <int DH>
size_t smem_bytes(int max_batch) {
  return Smem<DH>::TABLE_OFF + (size_t)(2 * max_batch + 2) * sizeof(int);
}

}  // namespace

int launch_attn_rows(space_ctx* ctx, const space_attn_args* a, const uint64_t* mask_rows,
                       cudaStream_t st) {
  const space_config& cfg = ctx->cfg;
  const int DH = cfg.head_dim;
  AttnPlanHost pl;
  plan(&cfg, ctx->sm_count, a->k, &pl);
  AttnParams p;
  memset(&p, 0, sizeof(p));
  p.B = a->batch; p.n_q = (a->k + 1) * (a->k + 1);
  p.H_q = cfg.n_q_heads; p.H_kv = cfg.n_kv_heads; p.G = p.H_q / p.H_kv;
  p.n_mblocks = pl.n_mblocks; p.rows_per_mb = pl.rows_per_mblock;
  p.n_groups = pl.n_ctas / pl.n_mblocks;
  p.out_dtype = a->out_dtype;
  p.s_cap = a->page_table ? (int64_t)a->pages_per_seq * SPACE_PAGE_SIZE : cfg.s_cap;
  p.page_table = a->page_table; p.pages_per_seq = a->pages_per_seq; p.n_pages = a->n_pages;
  p.scale_log2 = a->scale * 1.4426950408889634f;
  p.kv_len = a->kv_len; p.out = a->out; p.lse = a->lse; p.status = a->status;
  p.part = ctx->attn_part; p.err = ctx->counters + 3 * cfg.max_batch;
  p.desc = reinterpret_cast<int2*>(ctx->merge_cnt);
  p.owner = ctx->merge_cnt + (size_t)cfg.max_batch * cfg.n_kv_heads * 8 * 2;
  p.merge_by_owner = (a->batch * p.H_kv * p.n_mblocks > pl.n_ctas) ? 1 : 0;
  for (int i = 0; i < SPACE_MAX_ROWS; ++i) p.mask[i] = mask_rows[i];

  // TMA descriptors, rebuilt only when a base pointer or a stride changes
  const int64_t key[8] = {a->kv_stride_b, a->kv_stride_h, a->kv_stride_s, a->batch, p.n_q, -1,
                          a->page_table ? a->n_pages : 0, 0};
  if (ctx->tm_q_ptr != a->q || ctx->tm_k_ptr != a->k_cache || ctx->tm_v_ptr != a->v_cache ||
      memcmp(key, ctx->tm_key, sizeof(key)) != 0) {
    const cuuint64_t kd[4] = {(cuuint64_t)DH, (cuuint64_t)(a->page_table ? TILE_N : cfg.s_cap), (cuuint64_t)p.H_kv,
                              (cuuint64_t)(a->page_table ? a->n_pages : a->batch)};
    const cuuint64_t ks[3] = {(cuuint64_t)a->kv_stride_s * 2, (cuuint64_t)a->kv_stride_h * 2,
                              (cuuint64_t)a->kv_stride_b * 2};
    const cuuint32_t kb[4] = {64, TILE_N, 1, 1};
    const cuuint64_t qd[4] = {(cuuint64_t)DH, (cuuint64_t)p.H_q, (cuuint64_t)p.n_q, (cuuint64_t)a->batch};
    const cuuint64_t qs[3] = {(cuuint64_t)DH * 2, (cuuint64_t)p.H_q * DH * 2, (cuuint64_t)p.n_q * p.H_q * DH * 2};
    const cuuint32_t qb[4] = {64, (cuuint32_t)p.G, (cuuint32_t)(ROWS / p.G), 1};
    int rc = make_map((CUtensorMap*)ctx->tm_k, a->k_cache, kd, ks, kb);
    if (rc == SPACE_OK) rc = make_map((CUtensorMap*)ctx->tm_v, a->v_cache, kd, ks, kb);
    if (rc == SPACE_OK) rc = make_map((CUtensorMap*)ctx->tm_q, a->q, qd, qs, qb);
    if (rc != SPACE_OK) { ctx->tm_q_ptr = nullptr; return rc; }
    ctx->tm_q_ptr = a->q; ctx->tm_k_ptr = a->k_cache; ctx->tm_v_ptr = a->v_cache;
    memcpy(ctx->tm_key, key, sizeof(key));
  }
  memcpy(&p.tm_q, ctx->tm_q, sizeof(CUtensorMap));
  memcpy(&p.tm_k, ctx->tm_k, sizeof(CUtensorMap));
  memcpy(&p.tm_v, ctx->tm_v, sizeof(CUtensorMap));

  const int m_valid_max = p.rows_per_mb * p.G;
  const dim3 mgrid(p.merge_by_owner ? pl.n_ctas : a->batch * p.H_kv * p.n_mblocks, (m_valid_max * (DH / 4) + 127) / 128);
  if (DH == 128) {
    const size_t sm = smem_bytes<128>(cfg.max_batch);
    cudaFuncSetAttribute(attn_rows_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    {
      ProfScope ps(ctx, SPACE_K_ATTN, st);
      launch_pdl(attn_rows_kernel<128>, dim3(pl.n_ctas), dim3(THREADS), sm, st, p, cfg.max_batch);
    }
    {
      ProfScope ps(ctx, SPACE_K_MERGE, st);
      launch_pdl(attn_rows_merge_kernel<128>, mgrid, dim3(128), 0, st, p);
    }
  } else {
    const size_t sm = smem_bytes<64>(cfg.max_batch);
    cudaFuncSetAttribute(attn_rows_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    {
      ProfScope ps(ctx, SPACE_K_ATTN, st);
      launch_pdl(attn_rows_kernel<64>, dim3(pl.n_ctas), dim3(THREADS), sm, st, p, cfg.max_batch);
    }
    {
      ProfScope ps(ctx, SPACE_K_MERGE, st);
      launch_pdl(attn_rows_merge_kernel<64>, mgrid, dim3(128), 0, st, p);
    }
  }
  ctx->launches += 2;
  return cuda_ok(cudaGetLastError());
}
