// Tensor-core attention of the block rows over cache + block (Eq. 5) for sm_100a.
//
// Persistent split-KV flash-decode kernel.  The (sequence, kv head) key ranges
// are cut into 128-key tiles, the tiles of all sequences form one flat list
// and every thread-block group takes an equal contiguous share of it, so ragged
// batches balance without host knowledge of the lengths.  A share that does not
// cover a whole (sequence, head) leaves an unnormalised partial (reference
// maximum, sum, accumulator) in scratch memory; attn_merge_kernel combines the
// partials of every (sequence, head) that was cut.
//
// The query block of one kv head is small here (the (k+1)^2 block rows times the GQA
// group, at most 64 rows; wider blocks go to attn_rows.cu), so the two tile products are taken transposed: the
// 128 keys of a tile are the MMA M extent and the query rows the N extent,
//   S^T = K Q^T   (128 x N),      O^T += V^T (P_hi + P_lo)^T   (head_dim x N),
// which costs N/128 of a full tile and puts one key on every TMEM lane.
//
// Inside a block (12 warps):
//   warps 0, 2  stream K and V tiles with TMA into two rings of shared-memory
//           stages (a K stage is free once K Q^T has read it, a V stage once V^T P^T has)
//           (warp 0 also loads the query rows of each share, one share ahead)
//   warp 1  issues the S^T products (tcgen05.mma) into one of two TMEM buffers
//   warp 3  issues the O^T products
//   warps 4-11  two threads per key: read S^T from TMEM, apply the Eq. 5 mask
//           on tiles that touch the block or a share boundary, P = exp2(score -
//           reference) as two bf16 terms into shared memory for the second MMA.
//           The per-row reference is set on a share's first tile and moved only
//           when a score exceeds it by 2^60 (a block-wide vote per tile), so no
//           per-tile row maximum is needed; row sums are kept per key and added
//           across keys once per share.
// Every wait is bounded; an expired wait sets SPACE_ST_TIMEOUT and the block
// drains and exits.
//
// One sequence (the usual decoding case) takes a partition of its own: every kv head gets the
// same number of groups, piece i of a head takes tiles i, i + pieces, ... (so a group's first
// tile does not depend on the length and is requested, with the query rows, before the length
// is read), and the groups left over take the heads' last tiles, the ones with the block's own
// keys and the Eq. 5 mask.
#include "common.cuh"
#include "tc_common.cuh"
#include <cuda.h>
#include <math_constants.h>

namespace {

constexpr int TILE_N = 128;            // keys per tile
constexpr int SHARE_COST = 4;          // fixed cost of a share (query load, first tile, last product, epilogue) in tiles; swept 2..8
constexpr int ROWS = 128;              // MMA M
constexpr int THREADS = 384;            // K, MMA, V, Q warps + 8 softmax warps
constexpr uint64_t WAIT_NS = 1000000000ull;   // one second per wait

struct AttnParams {
  CUtensorMap tm_q, tm_k, tm_v;
  int B, n_q, H_q, H_kv, G;
  int n_mblocks, rows_per_mb;          // query-row blocks per kv head; block rows i per block
  int n_pad;                           // rows_per_mb * G rounded up to 16: N of the MMAs
  int n_groups;                        // thread-block groups (grid = n_groups * n_mblocks)
  int out_dtype;
  int spec;                            // one sequence: every group requests its first K tile before the length is read
  int64_t s_cap;                       // rows a sequence may hold (paged: pages_per_seq * SPACE_PAGE_SIZE)
  // Paged cache (page_table != nullptr): tm_k / tm_v describe a pool [n_pages][H_kv][TILE_N][d]; tile t
  // of sequence b is the whole page page_table[b * pages_per_seq + t].  No tile is shifted back then:
  // the last one may end in rows that belong to no key, whose scores are masked and whose V rows are
  // cleared in shared memory before the O^T product reads them.
  const int32_t* page_table; int pages_per_seq, n_pages;
  float scale_log2;                    // scale * log2(e)
  const int32_t* kv_len;
  void* out; float* lse; int32_t* status;
  float* part;                         // [slots][ROWS*(DH+2)]
  int* err;                            // one word: first timeout site
  int2* desc;                          // [B*H_kv*n_mblocks] {first partial slot, number of partials} of each cut
  int* owner;                          // [grid] (sequence, kv head) whose last piece this thread block computed, or -1
  int merge_by_owner;                  // the merge grid is indexed by attention thread block, not by (sequence, head)
  // Eq. 5 per (query column, block key), worked out by the host once per call: bit q of
  // visq[mb][j] says that query column q of query-row block mb (block row mb * rows_per_mb + q / G,
  // any of its G heads) sees block key j
  uint64_t visq[2][SPACE_MAX_ROWS];
};

// Page of tile t of sequence b (paged cache).  An entry outside the pool is flagged and answered
// with a page past the pool's end: the TMA load then fills the tile with zeros.
// (flag = false: a request made before the length is known, for a tile the sequence may not have.)
__device__ __forceinline__ int page_of(const AttnParams& p, int b, int t, bool flag = true) {
  const int pg = t < p.pages_per_seq ? p.page_table[(int64_t)b * p.pages_per_seq + t] : -1;
  if (pg >= 0 && pg < p.n_pages) return pg;
  if (flag && p.status) atomicOr(p.status + b, SPACE_ST_BAD_PAGE);
  return p.n_pages;
}

// One share: tiles t0, t0 + step, ... (n of them) of the T tiles of (sequence b, kv head h).
struct Seg {
  int b, h, t0, n, step, T, L, slot, dfirst, dn;   // slot: partial slot; dfirst/dn: cut (aligned mode)
  __device__ __forceinline__ int tile_at(int j) const { return t0 + j * step; }
};

// Optional per-block timeline (compiled in with -DSPACE_TIMELINE): one %globaltimer stamp
// per named point and thread block, read back with space_debug_timeline_read.
#ifdef SPACE_TIMELINE
#define TL_POINTS 16
__device__ unsigned long long g_timeline[256 * TL_POINTS];
#define TL(i) do { unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); \
                   g_timeline[blockIdx.x * TL_POINTS + (i)] = t_; } while (0)
// the same for the merge kernel: four points per thread block (entry, dependency wait returned,
// descriptor in registers, output stored), written by thread 0
__device__ unsigned long long g_timeline_merge[4096 * 4];
#define TLM(i) do { if (threadIdx.x == 0 && blockIdx.y * gridDim.x + blockIdx.x < 4096) { unsigned long long t_; \
                   asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); \
                   g_timeline_merge[(blockIdx.y * gridDim.x + blockIdx.x) * 4 + (i)] = t_; } } while (0)
#else
#define TL(i) do { } while (0)
#define TLM(i) do { } while (0)
#endif   // slot: partial slot; dfirst/dn: cut (aligned mode)

// PTX helpers: tc_common.cuh.  Every wait of this kernel is bounded by WAIT_NS.
using namespace tc;
__device__ __noinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* err, int site) {
  return mbar_wait_bounded(bar, parity, abort_flag, err, site, WAIT_NS, 64);   // sleeps between polls
}
__device__ __noinline__ void mbar_drain(uint32_t bar, uint32_t parity) { mbar_drain_bounded(bar, parity, WAIT_NS); }

// ------------------------------------------------------------ work partition
// Flat tile index space: sequence-major, then kv head, then tile.  Group g of
// n_groups owns flat tiles [W*g/n_groups, W*(g+1)/n_groups).
// floor(a * b / c) for a*b that may need 64 bits; 32-bit division when it fits
__device__ __forceinline__ long long muldiv(long long a, long long b, long long c) {
  const unsigned long long prod = (unsigned long long)a * (unsigned long long)b;
  if ((prod >> 32) == 0) return (long long)((unsigned)prod / (unsigned)c);
  return (long long)(prod / (unsigned long long)c);
}

// Piece `piece` of `a` of a (sequence, head) with T tiles: tiles [t0, t1).  When the last tile is a
// partial one and there are at least `a` full tiles, the full tiles are cut evenly (the first pieces
// take the remainder) and the partial tile goes to the last piece on top; otherwise all T tiles are
// cut evenly.
__device__ __forceinline__ void even_cut(int T, int n_keys, int a, int piece, int& t0, int& t1) {
  const int Tf = (n_keys % TILE_N) ? T - 1 : T;
  const int Tc = (Tf < T && a <= Tf) ? Tf : T;
  const int q = Tc / a, r = Tc - q * a;
  t0 = piece * q + min(piece, r);
  t1 = t0 + q + (piece < r ? 1 : 0);
  if (piece == a - 1) t1 = T;
}

struct Partition {
  const int* seq_len;    // [B]   verified length, or -1 for a sequence that does not fit
  const int* prefix;     // [B+1] flat offset of sequence b
  // aligned mode: {b, h, t0, n, T, L, first slot of the cut, pieces in the cut, step, early requests
  // serve the first share, head stride from share to share, slot (slots per head when the stride is
  // not 0), number of shares}
  const int* seg0;
  int B, H_kv, n_q, group, ngroups;
  long long cur, end;
  int b;
  bool aligned;
  // Flat mode: only min(n_groups, W) groups take part, so every taking-part group
  // owns at least one tile and the groups of one (sequence, head) are consecutive.
  // Aligned mode (few tiles per group): every (sequence, head) gets a whole number
  // of groups and is cut evenly among them, so no group straddles two of them and
  // pays the per-share set-up and epilogue twice.
  // agroups: groups that have a share in aligned mode, or < 0 for flat mode
  __device__ void init(const int* sl, const int* pf, int agroups, const int* seg0_, int B_, int H, int nq,
                       int group_, int n_groups) {
    seq_len = sl; prefix = pf; seg0 = seg0_; B = B_; H_kv = H; n_q = nq; b = 0;
    group = group_; ngroups = n_groups;
    aligned = agroups >= 0;
    if (aligned) {
      cur = 0; end = seg0_[12];
      return;
    }
    const long long W = pf[B_];
    const long long NG = W < n_groups ? W : n_groups;
    if (group_ >= NG) { cur = end = 0; return; }
    cur = muldiv(W, group_, NG);
    end = muldiv(W, group_ + 1, NG);
  }
  __device__ bool next(Seg& s) {
    if (aligned) {
      // the shares were worked out once per thread block during the set-up: one, or (one
      // sequence, groups left over after every head got its pieces) the last tile of several heads
      if (cur >= end) return false;
      const int4 u = reinterpret_cast<const int4*>(seg0)[0], v = reinterpret_cast<const int4*>(seg0)[1];
      s.b = u.x; s.h = u.y; s.t0 = u.z; s.n = u.w; s.T = v.x; s.L = v.y; s.dfirst = v.z; s.dn = v.w;
      s.step = seg0[8];
      s.slot = seg0[11];
      const int hstep = seg0[10];
      if (hstep > 0) {
        s.h = u.y + (int)cur * hstep;
        s.dfirst = s.h * seg0[11];
        s.slot = s.dfirst + seg0[11] - 1;
      }
      ++cur;
      return true;
    }
    // Flat mode: the list holds T + SHARE_COST entries per (sequence, head); the
    // first SHARE_COST stand for the fixed cost of starting a share there, so
    // that equal list shares are shares of about equal time.
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
      if (t1 <= t0) continue;                               // only the cost entries: no tiles here
      s.b = b; s.h = h; s.t0 = t0; s.n = t1 - t0; s.step = 1; s.T = T; s.L = L;
      s.slot = b * H_kv + h + group; s.dfirst = -1; s.dn = 0;
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

// Shared-memory plan (up to 64 query rows per thread block).
template <int DH>
struct Smem {
  static constexpr int HALVES = DH / 64;
  static constexpr int TILE_BYTES = TILE_N * DH * 2;         // one K or V tile
  static constexpr int Q_ROWS = 64;                          // query rows (with padding) per thread block
  static constexpr int Q_BYTES = Q_ROWS * DH * 2;
  static constexpr int P_PART = TILE_N * 128;                // P_hi or P_lo: [key][64 queries] bf16
  static constexpr int K_STAGES = (DH == 128) ? 2 : 3;
  static constexpr int V_STAGES = (DH == 128) ? 2 : 4;
  static constexpr int P_BUFS = 1;                           // P^T buffers (each P_hi + P_lo); a second one, so that the exponentials of a tile
                                                             // overlap the O^T product of the tile before, measured no faster
  static constexpr int RS = 64;                              // query rows (padded) per thread block at most
  static constexpr int Q_BUFS = 2;                           // query buffers: the next share's rows load early
  static constexpr int Q_OFF = 0;
  static constexpr int K_OFF = Q_BUFS * Q_BYTES;
  static constexpr int V_OFF = K_OFF + K_STAGES * TILE_BYTES;
  static constexpr int P_OFF = V_OFF + V_STAGES * TILE_BYTES;
  static constexpr int BAR_OFF = P_OFF + P_BUFS * 2 * P_PART;
  // q_full[2], q_empty[2], k_full[], k_empty[], v_full[], v_empty[], s_full[2], p_ready[2], pv_done[2], drain
  static constexpr int N_BARS = 4 + 2 * K_STAGES + 2 * V_STAGES + 6 + 1;
  static constexpr int MISC_OFF = BAR_OFF + (N_BARS * 8 + 15) / 16 * 16;   // tmem base, abort flag (16-byte aligned:
                                                                           // the float arrays below are read as float4)
  static constexpr int SEG0_OFF = MISC_OFF + 16;             // Seg of this group's only share (aligned mode)
  static constexpr int MREF_OFF = MISC_OFF + 96;             // [2][RS] float: reference maximum per query row
  static constexpr int XQ_OFF = MREF_OFF + 2 * RS * 4;       // [4 quarters][RS] float: cross-lane reductions
  static constexpr int FQ_OFF = XQ_OFF + 4 * RS * 4;         // [RS] float: rescale factors / final row sums
  static constexpr int VISQ_OFF = FQ_OFF + RS * 4;           // [64] uint64: query columns that see block key j (bit = column)
  static constexpr int TABLE_OFF = VISQ_OFF + SPACE_MAX_ROWS * 8;   // seq_len[max_batch], prefix[max_batch+1]
  // with the tables of the largest batch (128 sequences) the plan must fit the 227 KB a block may have
  static_assert(TABLE_OFF + (2 * 128 + 1) * 4 <= 227 * 1024, "shared-memory plan too large");
};

// Barrier over the 256 softmax threads (id 1); the second form also ORs a predicate.
__device__ __forceinline__ void soft_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ bool soft_any(bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %1, 0;\n\t"
      "bar.red.or.pred q, 1, 256, p;\n\tselp.b32 %0, 1, 0, q;\n\t}"
      : "=r"(r) : "r"((uint32_t)pred) : "memory");
  return r != 0;
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// Instruction descriptor: bf16 x bf16 -> f32, M = 128, N = n; a_mn / b_mn = operand is MN-major.
__device__ __forceinline__ uint32_t instr_desc_rt(int n, int a_mn, int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(ROWS >> 4) << 24);
}

// ---- parts of the softmax threads that are off the hot path; kept out of line
// so that the per-tile loop stays small enough for the instruction cache ----
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t* r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t* r) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}

// Maximum over the 32 keys of this warp for each of 8 query rows (visible
// entries only); lane 0 stores them at dst[0..7].
__device__ __noinline__ void piece_key_max(uint32_t taddr, uint32_t vis, float* dst) {
  uint32_t sr[8];
  tmem_ld8(taddr, sr);
  tmem_wait_ld();
  float out[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    // order-preserving map float -> int so that one integer warp reduction does it
    const int bits = ((vis >> e) & 1u) ? (int)sr[e] : (int)0xFF800000u;      // -inf when not visible
    const int key = bits ^ ((bits >> 31) & 0x7FFFFFFF);
    const int mx = __reduce_max_sync(0xFFFFFFFFu, key);
    out[e] = __int_as_float(mx ^ ((mx >> 31) & 0x7FFFFFFF));
  }
  if ((threadIdx.x & 31) == 0) {
    reinterpret_cast<float4*>(dst)[0] = make_float4(out[0], out[1], out[2], out[3]);
    reinterpret_cast<float4*>(dst)[1] = make_float4(out[4], out[5], out[6], out[7]);
  }
}

// New reference for 8 query rows from the four quarter maxima in xq (rs floats apart); writes the
// reference to mnew[0..7] and (unless this is a share's first tile) the factor
// old -> new to fq[0..7].  Every thread that owns the rows computes the same
// values (identical writes).  All pointers are 16-byte aligned.
__device__ __noinline__ void piece_new_reference(const float* xq, int rs, const float* mold, float* mnew, float* fq,
                                                 float c, bool first) {
#pragma unroll
  for (int v = 0; v < 2; ++v) {
    const float4 a = reinterpret_cast<const float4*>(xq)[v], b = reinterpret_cast<const float4*>(xq + rs)[v];
    const float4 d = reinterpret_cast<const float4*>(xq + 2 * rs)[v], e = reinterpret_cast<const float4*>(xq + 3 * rs)[v];
    float tm[4] = {fmaxf(fmaxf(a.x, b.x), fmaxf(d.x, e.x)) * c, fmaxf(fmaxf(a.y, b.y), fmaxf(d.y, e.y)) * c,
                   fmaxf(fmaxf(a.z, b.z), fmaxf(d.z, e.z)) * c, fmaxf(fmaxf(a.w, b.w), fmaxf(d.w, e.w)) * c};
    float mo[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
    if (!first) {
      const float4 o = reinterpret_cast<const float4*>(mold)[v];
      mo[0] = o.x; mo[1] = o.y; mo[2] = o.z; mo[3] = o.w;
    }
    float mn[4], f[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (!(tm[j] > -CUDART_INF_F)) tm[j] = -CUDART_INF_F;  // also catches NaN
      mn[j] = fmaxf(mo[j], tm[j]);
      f[j] = (mo[j] > -CUDART_INF_F) ? fast_exp2(mo[j] - mn[j]) : 0.f;
    }
    reinterpret_cast<float4*>(mnew)[v] = make_float4(mn[0], mn[1], mn[2], mn[3]);
    if (!first) reinterpret_cast<float4*>(fq)[v] = make_float4(f[0], f[1], f[2], f[3]);
  }
}

// O^T[lane][8 columns] *= fq[0..7]
__device__ __noinline__ void piece_rescale(uint32_t taddr, const float* fq) {
  uint32_t o[8];
  tmem_ld8(taddr, o);
  tmem_wait_ld();
#pragma unroll
  for (int e = 0; e < 8; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * fq[e]);
  tmem_st8(taddr, o);
  tmem_wait_st();
}

// Warp roles
constexpr int WARP_K = 0, WARP_MMA = 1, WARP_V = 2, WARP_PV = 3, WARP_SOFTMAX0 = 4;
constexpr int L2_AHEAD_TILES = 1;      // tiles per operand a block asks L2 for before its dependency wait (more of them
                                       // crowd out the kernels that still run: measured slower)
constexpr float OVER_THRESHOLD = 60.f;   // re-reference a query row when a score exceeds its reference by 2^60

// The tile products are taken transposed: S^T = K Q^T (128 keys x N query rows)
// and O^T += V^T P^T (head_dim x N), so the MMA N extent is the number of
// query rows rounded up to 16 instead of a full 128-row tile, and one thread
// owns one key of the tile (all 128 TMEM lanes carry work).
// PAGED: the cache is a pool of pages behind a page table (see AttnParams); a build of its own, so
// that the contiguous form carries none of it (registers are at the limit of 384 threads).
template <int DH, bool PAGED>
__global__ void __launch_bounds__(THREADS, 1) attn_tc_kernel(const __grid_constant__ AttnParams p,
                                                             int max_batch) {
  using S = Smem<DH>;
  extern __shared__ __align__(1024) unsigned char sm[];
  const uint32_t sm_base = smem_u32(sm);
  const uint32_t bar0 = sm_base + S::BAR_OFF;
  auto BAR = [&](int i) { return bar0 + 8u * i; };
  constexpr int B_QFULL = 0, B_QEMPTY = 2, B_KFULL = 4, B_KEMPTY = B_KFULL + S::K_STAGES,
                B_VFULL = B_KEMPTY + S::K_STAGES, B_VEMPTY = B_VFULL + S::V_STAGES,
                B_SFULL = B_VEMPTY + S::V_STAGES, B_PREADY = B_SFULL + 2, B_PVDONE = B_SFULL + 4,
                B_DRAIN = B_SFULL + 6;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + S::MISC_OFF);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + S::MISC_OFF + 4);
  float* mref_buf = reinterpret_cast<float*>(sm + S::MREF_OFF);
  float* xq = reinterpret_cast<float*>(sm + S::XQ_OFF);
  float* fq = reinterpret_cast<float*>(sm + S::FQ_OFF);
  uint64_t* visq = reinterpret_cast<uint64_t*>(sm + S::VISQ_OFF);
  int* seq_len = reinterpret_cast<int*>(sm + S::TABLE_OFF);
  int* prefix = seq_len + max_batch;
  volatile int* agroups = reinterpret_cast<volatile int*>(sm + S::MISC_OFF + 8);
  int* seg0 = reinterpret_cast<int*>(sm + S::SEG0_OFF);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int group = blockIdx.x / p.n_mblocks, mb = blockIdx.x % p.n_mblocks;
  const int i0 = mb * p.rows_per_mb;                       // first block row of this query-row block
  // query rows (block row, head) handled here: 0 .. m_valid-1; N of the MMAs is n_pad
  const int m_valid = min(p.rows_per_mb, p.n_q - i0) * p.G;
  const int n_pad = p.n_pad;

  // ---- set-up ------------------------------------------------------------
  pdl_launch_dependents();
  if (threadIdx.x == 0) TL(0);
  if (threadIdx.x == 0) {
    *abort_flag = (sm_base & 1023u) ? 1 : 0;               // swizzled tiles need a 1024-byte aligned base
    for (int i = 0; i < 2; ++i) { mbar_init(BAR(B_QFULL + i), 1); mbar_init(BAR(B_QEMPTY + i), 1); }
    for (int s = 0; s < S::K_STAGES; ++s) { mbar_init(BAR(B_KFULL + s), 1); mbar_init(BAR(B_KEMPTY + s), 1); }
    for (int s = 0; s < S::V_STAGES; ++s) { mbar_init(BAR(B_VFULL + s), 1); mbar_init(BAR(B_VEMPTY + s), 1); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(BAR(B_SFULL + i), 1);
      mbar_init(BAR(B_PREADY + i), 256);
    }
    mbar_init(BAR(B_PVDONE), 1);
    mbar_init(BAR(B_PVDONE + 1), 1);
    mbar_init(BAR(B_DRAIN), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == WARP_MMA) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (warp >= WARP_SOFTMAX0 && threadIdx.x - WARP_SOFTMAX0 * 32 < SPACE_MAX_ROWS) {
    // this block's visibility words into shared memory (the softmax threads index them by key)
    const int j = threadIdx.x - WARP_SOFTMAX0 * 32;
    visq[j] = p.visq[mb][j];
  }
  // single-sequence partition (explained where the tables are built, below)
  const int sp_base = max(p.n_groups / p.H_kv, 1), sp_extra = p.n_groups - sp_base * p.H_kv;
  const bool sp_helper = group >= sp_base * p.H_kv;
  const int sp_h = sp_helper ? group - sp_base * p.H_kv : group / sp_base;
  const int sp_piece = sp_helper ? 0 : group - sp_h * sp_base;
  const bool early = p.spec && !sp_helper;                 // this group requests Q and its first K tile at once
  if (warp == WARP_K && lane == 0)
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&p.tm_k) : "memory");
  if (warp == WARP_V && lane == 0)
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&p.tm_v) : "memory");
  if (warp == WARP_MMA && lane == 0)
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&p.tm_q) : "memory");
  if (early && !PAGED && lane == 0 && (warp == WARP_K || warp == WARP_V)) {
    // A regular group's tiles (sp_piece, sp_piece + sp_base, ...) of head sp_h do not depend on the
    // length, so L2 is asked for them now, while the kernel before this one may still be running:
    // with a programmatic launch this block is resident long before its dependency wait returns,
    // and the tile loads after the wait then find their lines in L2 instead of paying the DRAM
    // latency in a burst of all blocks at once.  Only a request to the cache: whatever the earlier
    // kernel still writes is what the loads will see.  The length is read here as a hint for how
    // many tiles are worth asking for (a stale value costs or saves a request, never an error).
    const uint64_t pol = l2_evict_first_policy();
    const int Lh = *reinterpret_cast<const volatile int*>(p.kv_len);
    const int Th = (Lh >= 0 && (int64_t)Lh + p.n_q <= p.s_cap) ? (Lh + p.n_q) / TILE_N : 0;   // whole tiles
    const CUtensorMap* tm = warp == WARP_K ? &p.tm_k : &p.tm_v;
    for (int j = 0, t = sp_piece; j < L2_AHEAD_TILES && t < Th; ++j, t += sp_base) {
#pragma unroll
      for (int hf = 0; hf < S::HALVES; ++hf) tma_prefetch_l2_4d(tm, hf * 64, t * TILE_N, sp_h, 0, pol);
    }
  }
  // barriers and the TMEM allocation are visible to every warp before the first
  // global access (with a programmatic launch this part runs under the previous kernel)
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (threadIdx.x == 0) TL(1);
  pdl_wait();                                              // global memory from here on
  if (threadIdx.x == 0) TL(2);
  const bool single = p.B == 1;
  // One sequence, no more kv heads than groups: every head gets `base` groups (piece i of a head
  // takes tiles i, i + base, ...: its first tile does not depend on the length), and the groups
  // left over are helpers that each take the last tile of some heads -- the one with the block's
  // own keys, whose Eq. 5 mask makes it the slowest -- so that no regular piece carries it on top
  // of its share of the full tiles.
  if (early && warp == WARP_K && lane == 0 && !*abort_flag) {
    // Which head and which first tile a regular group works on does not depend on the length,
    // so its query rows and its first K tile are requested before the length is even read (one
    // memory round trip earlier).  Should the length turn out too short for that tile, the S^T
    // issuer lets both buffers go unused.
    mbar_expect_tx(BAR(B_QFULL), (uint32_t)n_pad * DH * 2);
#pragma unroll
    for (int hf = 0; hf < S::HALVES; ++hf)
      tma_load_4d(sm_base + S::Q_OFF + hf * (n_pad * 128), &p.tm_q, BAR(B_QFULL), hf * 64, sp_h * p.G, i0, 0);
    mbar_expect_tx(BAR(B_KFULL), S::TILE_BYTES);
#pragma unroll
    for (int hf = 0; hf < S::HALVES; ++hf)
      tma_load_4d_hint(sm_base + S::K_OFF + hf * (TILE_N * 128), &p.tm_k, BAR(B_KFULL), hf * 64,
                       PAGED ? 0 : sp_piece * TILE_N, sp_h, PAGED ? page_of(p, 0, sp_piece, false) : 0,
                       l2_evict_first_policy());
    TL(3);
  }
  if (single) {
    // One sequence (the usual decoding case): the tables have a closed form, so every
    // thread works them out for itself from the one length (identical values, each
    // thread reads back what it wrote) and no warp has to hand them over.
    const int L0 = p.kv_len[0];
    const bool okL = L0 >= 0 && (int64_t)L0 + p.n_q <= p.s_cap;
    if (!okL && blockIdx.x == 0 && threadIdx.x == 0 && p.status) atomicOr(p.status, SPACE_ST_CAPACITY);
    const int L = okL ? L0 : -1;
    const int T = okL ? (L + p.n_q + TILE_N - 1) / TILE_N : 0;
    if (threadIdx.x == 0 && L0 != 0x7FFFFFFF) TL(14);
    seq_len[0] = L; prefix[0] = 0; prefix[1] = okL ? (T + SHARE_COST) * p.H_kv : 0;
    int ag = -1, spec_ok = 0;
    const int W = T * p.H_kv;
    const bool cut_aligned = W > 0 && W < 8 * p.n_groups && p.H_kv <= p.n_groups;
    const bool helpers = cut_aligned && sp_extra > 0 && T > sp_base;   // the last tile goes to a helper group
    if (p.spec && sp_helper && helpers) {
      // A helper knows its first share as soon as it has the length: the last tile of head sp_h.
      // Its query rows and that tile are requested here, ahead of the tables and the producer's
      // own start-up, which would come a microsecond later.
      spec_ok = 1;
      if (warp == WARP_K && lane == 0 && !*abort_flag) {
        const int n_keys = L + p.n_q;
        const int kt = PAGED ? 0 : ((T * TILE_N <= n_keys) ? (T - 1) * TILE_N : n_keys - TILE_N);
        const int kb = PAGED ? page_of(p, 0, T - 1) : 0;
        mbar_expect_tx(BAR(B_QFULL), (uint32_t)n_pad * DH * 2);
#pragma unroll
        for (int hf = 0; hf < S::HALVES; ++hf)
          tma_load_4d(sm_base + S::Q_OFF + hf * (n_pad * 128), &p.tm_q, BAR(B_QFULL), hf * 64, sp_h * p.G, i0, 0);
        mbar_expect_tx(BAR(B_KFULL), S::TILE_BYTES);
#pragma unroll
        for (int hf = 0; hf < S::HALVES; ++hf)
          tma_load_4d_hint(sm_base + S::K_OFF + hf * (TILE_N * 128), &p.tm_k, BAR(B_KFULL), hf * 64, kt, sp_h, kb,
                           l2_evict_first_policy());
        TL(3);
      }
    }
    if (cut_aligned) {
      ag = p.n_groups;
      const int Treg = helpers ? T - 1 : T;                // tiles cut among the regular pieces
      const int dn = helpers ? sp_base + 1 : min(sp_base, T);
      if (!sp_helper) {
        const int n_mine = sp_piece < Treg ? (Treg - sp_piece + sp_base - 1) / sp_base : 0;
        spec_ok = (n_mine > 0 && (sp_piece + 1) * TILE_N <= L + p.n_q) ? 1 : 0;   // the requested tile is this share's first
        if (PAGED && spec_ok && warp == WARP_K && lane == 0) (void)page_of(p, 0, sp_piece);   // flags a bad entry
        reinterpret_cast<int4*>(seg0)[0] = make_int4(0, sp_h, sp_piece, n_mine);
        reinterpret_cast<int4*>(seg0)[1] = make_int4(T, L, sp_h * (sp_base + 1), dn);
        seg0[8] = sp_base; seg0[10] = 0; seg0[11] = sp_h * (sp_base + 1) + sp_piece; seg0[12] = n_mine > 0 ? 1 : 0;
      } else {
        // helper e: the last tile of heads e, e + extra, e + 2 extra, ...
        reinterpret_cast<int4*>(seg0)[0] = make_int4(0, sp_h, T - 1, 1);
        reinterpret_cast<int4*>(seg0)[1] = make_int4(T, L, 0, dn);
        seg0[8] = 1; seg0[10] = sp_extra; seg0[11] = sp_base + 1;
        seg0[12] = helpers ? (p.H_kv - sp_h + sp_extra - 1) / sp_extra : 0;
      }
    }
    seg0[9] = spec_ok;
    *agroups = ag;
  } else if (warp == WARP_SOFTMAX0) {
    // per-sequence tile counts and their running sum, 32 sequences per round
    int carry = 0, nvalid = 0;
    for (int b0 = 0; b0 < p.B; b0 += 32) {
      const int b = b0 + lane;
      int L = -1, tiles = 0;
      bool ok = false;
      if (b < p.B) {
        L = p.kv_len[b];
        ok = L >= 0 && (int64_t)L + p.n_q <= p.s_cap;
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
      nvalid += __popc(__ballot_sync(0xFFFFFFFFu, ok));
    }
    // aligned mode when a group would get fewer than 8 tiles: groups per (sequence,
    // head) a_b = floor(groups * T_b / W), at least 1 tile each; fall back to the flat
    // cut if that needs more groups than there are
    if (lane == 0) { seg0[8] = 1; seg0[9] = 0; seg0[10] = 0; seg0[11] = group; seg0[12] = 0; }   // no share yet
    __syncwarp();
    const int Wv = carry;                                  // list entries (tiles + share costs)
    const int W = Wv - SHARE_COST * p.H_kv * nvalid;       // real tiles
    int acarry = -1;
    if (W > 0 && W < 8 * p.n_groups) {
      acarry = 0;
      for (int b0 = 0; b0 < p.B; b0 += 32) {
        const int b = b0 + lane;
        int a = 0, T = 0, L = -1;
        if (b < p.B) L = seq_len[b];                         // written by this lane above
        if (L >= 0) {
          T = (L + p.n_q + TILE_N - 1) / TILE_N;
          a = (int)muldiv(p.n_groups, T, W);
          a = max(1, min(a, T));
        }
        int incl = a * p.H_kv;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
          if (lane >= o) incl += v;
        }
        const int first = acarry + incl - a * p.H_kv;        // first group of sequence b
        if (a > 0 && group >= first && group < first + a * p.H_kv) {
          // this group's share: head h, piece `piece` of a (see even_cut)
          const int local = group - first;
          const int h = local / a, piece = local - h * a;
          int t0, t1;
          even_cut(T, L + p.n_q, a, piece, t0, t1);
          reinterpret_cast<int4*>(seg0)[0] = make_int4(b, h, t0, t1 - t0);
          reinterpret_cast<int4*>(seg0)[1] = make_int4(T, L, first + h * a, a);
          seg0[12] = 1;
        }
        acarry += __shfl_sync(0xFFFFFFFFu, incl, 31);
      }
      if (acarry > p.n_groups) acarry = -1;
    }
    if (lane == 0) {
      prefix[p.B] = Wv;
      *agroups = acarry;
    }
  }
  if (!single) __syncthreads();                            // the tables of warp 4 reach every warp
  const uint32_t tmem = *tmem_slot;
  // TMEM columns: S^T buffers at 0 and 128 (n_pad <= 128 columns each), [O_hi^T | O_lo^T] at 256
  // (64 columns each)
  const uint32_t TM_S0 = tmem, TM_O = tmem + 256;

  Partition part;
  part.init(seq_len, prefix, *agroups, seg0, p.B, p.H_kv, p.n_q, group, p.n_groups);
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
      // Early requests (one sequence): when this share's first tile is the requested one, the K
      // producer skips the query rows and that tile; when it is not, the two buffers are given
      // back by the S^T issuer and the rings start one slot further.
      if (is_k) TL(15);
      const uint64_t kv_policy = l2_evict_first_policy();
      bool pre = p.spec && is_k && seg0[9] != 0;           // Q and the first K tile of the first share are on their way
      const uint32_t koff = (early && is_k && !pre) ? 1u : 0u;
      uint32_t gt = 0, seg = koff;
      bool ok = true;
      const uint32_t q_bytes = (uint32_t)n_pad * DH * 2;
      // The very first S^T product needs only Q and the first K tile: V holds back
      // until that K tile has landed, so that it does not share the opening burst.
      bool v_hold = !is_k;
      while (ok && part.next(sg)) {
        const int n_keys = sg.L + p.n_q;
        if (is_k) {
          // the K producer also loads this share's query rows, into the buffer that
          // the share before the previous one used (with one buffer: the previous one)
          const uint32_t qb = seg % S::Q_BUFS, use = seg / S::Q_BUFS;
          if (!pre) {
            if (use > 0) ok = mbar_wait(BAR(B_QEMPTY + qb), (use - 1) & 1, abort_flag, p.err, 3);
            if (!ok) break;
            if (seg == 0) TL(3);
            mbar_expect_tx(BAR(B_QFULL + qb), q_bytes);
#pragma unroll
            for (int hf = 0; hf < S::HALVES; ++hf)
              tma_load_4d(sm_base + S::Q_OFF + qb * S::Q_BYTES + hf * (n_pad * 128), &p.tm_q, BAR(B_QFULL + qb),
                          hf * 64, sg.h * p.G, i0, sg.b);
          }
          ++seg;
        }
        for (int j = 0; j < sg.n && ok; ++j, ++gt) {
          if (pre) { pre = false; continue; }                 // requested before the length was known
          const int t = sg.tile_at(j);
          const uint32_t g = gt + koff;
          const int s = g % n_st;
          if (g >= (uint32_t)n_st)
            ok = mbar_wait(BAR(b_empty + s), ((g / n_st) - 1) & 1, abort_flag, p.err, is_k ? 1 : 2);
          if (!ok) break;
          if (v_hold || (is_k && g == 1)) {                 // (the second K tile holds back as well)
            ok = mbar_wait(BAR(B_KFULL), 0, abort_flag, p.err, 14);
            v_hold = false;
            if (!ok) break;
          }
          // the last tile of a sequence is shifted back so that it ends at the
          // last key: rows past the end are never read (they may hold anything)
          // (a paged cache has whole pages for tiles instead; see AttnParams)
          const int kt = PAGED ? 0 : (((t + 1) * TILE_N <= n_keys) ? t * TILE_N : n_keys - TILE_N);
          const int kb = PAGED ? page_of(p, sg.b, t) : sg.b;
          const uint32_t dst = ring + s * S::TILE_BYTES;
          mbar_expect_tx(BAR(b_full + s), S::TILE_BYTES);
#pragma unroll
          for (int hf = 0; hf < S::HALVES; ++hf)
            tma_load_4d_hint(dst + hf * (TILE_N * 128), tm, BAR(b_full + s), hf * 64, kt, sg.h, kb, kv_policy);
          if (is_k) TL(7);
        }
      }
      // drain: every issued copy must have landed before the block may exit
      const uint32_t issued = gt + koff;
      const uint32_t first = issued > (uint32_t)n_st ? issued - n_st : 0;
      for (uint32_t g = first; g < issued; ++g) mbar_drain(BAR(b_full + g % n_st), (g / n_st) & 1);
      if (is_k && seg > 0) {
        mbar_drain(BAR(B_QFULL + (seg - 1) % S::Q_BUFS), ((seg - 1) / S::Q_BUFS) & 1);
        if (S::Q_BUFS == 2 && seg > 1) mbar_drain(BAR(B_QFULL + (seg - 2) % 2), ((seg - 2) / 2) & 1);
      }
    }
  } else if (warp == WARP_MMA) {
    // ================= S^T issuer ==========================================
    if (lane == 0) {
      const uint32_t idesc_qk = instr_desc_rt(n_pad, 0, 0);   // A = K tile (K-major), B = Q (K-major)
      // descriptors of the first stage of every operand; a later stage or k-step
      // only adds to the 14-bit address field (16-byte units, no carry possible)
      const uint64_t kdesc0 = smem_desc(sm_base + S::K_OFF, 16, 1024);           // K-major rows of 128 bytes
      const uint64_t qdesc0 = smem_desc(sm_base + S::Q_OFF, 16, 1024);
      uint32_t gt = 0, seg = 0, koff = 0;
      bool ok = true;
      if (early && seg0[9] == 0) {
        // the early requests do not serve this group's first share: once they have landed their
        // buffers go back to the producer unused
        ok = mbar_wait(BAR(B_QFULL), 0, abort_flag, p.err, 15);
        if (ok) ok = mbar_wait(BAR(B_KFULL), 0, abort_flag, p.err, 16);
        mbar_arrive(BAR(B_QEMPTY));
        mbar_arrive(BAR(B_KEMPTY));
        seg = 1; koff = 1;
      }
      while (ok && part.next(sg)) {
        const uint32_t qb = seg % S::Q_BUFS, use = seg / S::Q_BUFS;
        if (gt == 0) TL(12);
        ok = mbar_wait(BAR(B_QFULL + qb), use & 1, abort_flag, p.err, 6);
        const uint64_t qd = qdesc0 + (uint64_t)((qb * S::Q_BYTES) >> 4);
        const int n = sg.n;
        for (int j = 0; j < n && ok; ++j, ++gt) {
          const int s = (gt + koff) % S::K_STAGES, buf = gt & 1;
          ok = mbar_wait(BAR(B_KFULL + s), ((gt + koff) / S::K_STAGES) & 1, abort_flag, p.err, 7);
          if (gt == 0) TL(4);
          // S^T buffer `buf` was last read by the softmax of tile gt-2
          if (ok && gt >= 2) ok = mbar_wait(BAR(B_PREADY + buf), ((gt - 2) >> 1) & 1, abort_flag, p.err, 8);
          if (!ok) break;
          tc_fence_after();
          const uint64_t kd = kdesc0 + (uint64_t)((s * S::TILE_BYTES) >> 4);
#pragma unroll
          for (int kk = 0; kk < DH / 16; ++kk) {
            // 64-wide half of d, then 32 bytes per 16 elements inside the swizzled row
            const uint32_t koff = (kk >> 2) * (TILE_N * 128) + (kk & 3) * 32;
            const uint32_t qoff = (kk >> 2) * (n_pad * 128) + (kk & 3) * 32;
            mma_ss(TM_S0 + buf * 128, kd + (uint64_t)(koff >> 4), qd + (uint64_t)(qoff >> 4), idesc_qk,
                   kk > 0 ? 1u : 0u);
          }
          tc_commit(BAR(B_SFULL + buf));
          tc_commit(BAR(B_KEMPTY + s));
          if (j == n - 1) tc_commit(BAR(B_QEMPTY + qb));
        }
        ++seg;
      }
    }
  } else if (warp == WARP_PV) {
    // ================= O^T issuer ===========================================
    // A thread of its own: the S^T products of the next tile need not queue
    // behind the sixteen instructions of this one.
    if (lane == 0) {
      // B = [P_hi | P_lo]: the two 64-column blocks lie one leading-dimension stride
      // apart, so a single product of N = 128 gives O_hi^T in columns 0..63 and
      // O_lo^T in columns 64..127 (an instruction costs the same at every N here);
      // the epilogue adds the two.  Columns past the padded query rows hold whatever
      // the shared memory held; they only reach output columns nobody reads.
      const uint32_t idesc_pv = instr_desc_rt(128, 1, 1);   // A = V^T (d contiguous), B = P^T (queries contiguous)
      // V^T and P^T: 64-wide blocks TILE_N*128 bytes apart, 8-key groups 1024 bytes apart
      static_assert(S::P_PART == TILE_N * 128, "P_lo must follow P_hi at the block stride");
      const uint64_t vdesc0 = smem_desc(sm_base + S::V_OFF, TILE_N * 128, 1024);
      const uint64_t pdesc0 = smem_desc(sm_base + S::P_OFF, TILE_N * 128, 1024);
      uint32_t g = 0;
      bool ok = true;
      while (ok && part.next(sg)) {
        for (int j = 0; j < sg.n && ok; ++j, ++g) {
          const int s = g % S::V_STAGES;
          ok = mbar_wait(BAR(B_VFULL + s), (g / S::V_STAGES) & 1, abort_flag, p.err, 4);
          if (ok) ok = mbar_wait(BAR(B_PREADY + (g & 1)), (g >> 1) & 1, abort_flag, p.err, 5);
          if (!ok) break;
          tc_fence_after();
          const uint64_t ad0 = vdesc0 + (uint64_t)((s * S::TILE_BYTES) >> 4);
          const uint64_t pd0 = pdesc0 + (uint64_t)(((g % S::P_BUFS) * 2 * S::P_PART) >> 4);
#pragma unroll
          for (int kk = 0; kk < TILE_N / 16; ++kk) {
            // 16 keys further = 2048 bytes further in both operands; the first
            // product of a share overwrites O^T
            mma_ss(TM_O, ad0 + (uint64_t)((kk * 2048) >> 4), pd0 + (uint64_t)((kk * 2048) >> 4), idesc_pv,
                   (j == 0 && kk == 0) ? 0u : 1u);
          }
          tc_commit(BAR(B_VEMPTY + s));
          tc_commit(BAR(B_PVDONE + (g & 1)));
        }
      }
      // all tensor work done before TMEM is released (every S^T product was
      // consumed by the softmax before the O^T product that follows it)
      tc_commit(BAR(B_DRAIN));
      mbar_drain(BAR(B_DRAIN), 0);
    }
  } else {
    // ================= softmax / epilogue ==================================
    // One key of the tile per TMEM lane; two threads per key, each with one half
    // of the query-row columns, handled in pieces of 8 columns.
    constexpr int MAXP = 4;                                // pieces per thread at most
    const int quarter = warp & 3;                          // TMEM lane quarter this warp may touch
    const int half = (warp - WARP_SOFTMAX0) >> 2;
    const int kl = quarter * 32 + lane;                    // key within the tile; head-dim index in the epilogue
    const int sidx = half * 128 + kl;                      // index among the 256 softmax threads
    const int ncol = n_pad >> 1, col0 = half * ncol, np = ncol >> 3;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const float c = p.scale_log2;
    const uint32_t prow = sm_base + S::P_OFF + kl * 128;   // this key's 128-byte row in each P block
    const uint32_t swz = (uint32_t)(kl & 7);
    float lsum[MAXP][8];                                   // this key's share of every row sum
    float sv[MAXP][8];                                     // scores, then score - reference (log2 units)
    uint32_t gt = 0;
    int mpar = 0;                                          // which copy of the references is current
    const float* mref = mref_buf;
    // A failed (expired) wait does not leave the loops: every thread keeps the
    // same control flow so that the block-wide barriers below always match up;
    // once the abort flag is set all later waits return at once and the block drains.
    bool ok = true;
    int own = -1;                                          // item whose last piece of a cut this block holds
    while (part.next(sg)) {
      const int n_keys = sg.L + p.n_q;
#pragma unroll
      for (int j = 0; j < MAXP; ++j)
#pragma unroll
        for (int e = 0; e < 8; ++e) lsum[j][e] = 0.f;
      for (int jt = 0; jt < sg.n; ++jt, ++gt) {
        const int t = sg.tile_at(jt);
        const int buf = gt & 1;
        const bool first = (jt == 0);
        ok &= mbar_wait(BAR(B_SFULL + buf), (gt >> 1) & 1, abort_flag, p.err, 9);
        tc_fence_after();
        if (sidx == 0) { if (gt == 0) TL(5); TL(8); }
        const uint32_t ts = TM_S0 + buf * 128 + lane_addr + col0;
        // this key's scores for its columns, all loads in flight together
#pragma unroll
        for (int j = 0; j < MAXP; ++j)
          if (j < np) tmem_ld8(ts + j * 8, reinterpret_cast<uint32_t*>(sv[j]));
        tmem_wait_ld();
        const int lo = t * TILE_N;
        const int kt = (PAGED || (t + 1) * TILE_N <= n_keys) ? lo : n_keys - TILE_N;
        const int key = kt + kl;
        const int jb = key - sg.L;                         // block key index when >= 0
        // Visibility of this thread's key: keys before `lo` belong to the previous
        // tile; cached keys are seen by every row; block keys by the Eq. 5 mask.
        const bool masked = (kt + TILE_N > sg.L) || (kt < lo);   // same for the whole block
        uint64_t vis = ~0ull;
        if (masked) {
          if (key < lo) vis = 0ull;
          else if (jb >= p.n_q) vis = 0ull;                 // (paged cache) a row of the page past the last key
          else if (jb >= 0) vis = visq[jb] >> col0;         // (bits past this thread's columns are never looked at)
        }
        // ---- first tile of a share: references from scores at hand.  Any reference within
        // 2^60 of the row maximum is as good as the maximum itself (P keeps its relative
        // precision as P_hi + P_lo, sums are fp32); pass 0 below checks exactly that bound.
        // Every row sees every cached key, so the scores of the tile's first cached key that
        // counts serve all rows.  A tile without one holds block keys only (it is then the last
        // tile of its sequence): a row's own key is always visible to it (Eq. 5) and gives its
        // reference; rows before the tile's first block key see nothing here and get -inf.
        if (first) {
          float* mnew = mref_buf + (mpar ^ 1) * S::RS;
          const int vstart = max(kt, lo);                    // first key of the tile that counts
          if (vstart < sg.L) {
            if (key == vstart) {
#pragma unroll
              for (int j = 0; j < MAXP; ++j) {
                if (j < np) {
                  float4* dst = reinterpret_cast<float4*>(mnew + col0 + j * 8);
                  dst[0] = make_float4(sv[j][0] * c, sv[j][1] * c, sv[j][2] * c, sv[j][3] * c);
                  dst[1] = make_float4(sv[j][4] * c, sv[j][5] * c, sv[j][6] * c, sv[j][7] * c);
                }
              }
            }
          } else {
            // block keys only: every thread parks its raw scores in the P buffer (idle until pass 1
            // of this very tile), then one thread per query column fetches the score of that
            // row's own key
            float* stage = reinterpret_cast<float*>(sm + S::P_OFF) + kl * 64 + col0;
#pragma unroll
            for (int j = 0; j < MAXP; ++j) {
              if (j < np) {
                reinterpret_cast<float4*>(stage + j * 8)[0] = make_float4(sv[j][0], sv[j][1], sv[j][2], sv[j][3]);
                reinterpret_cast<float4*>(stage + j * 8)[1] = make_float4(sv[j][4], sv[j][5], sv[j][6], sv[j][7]);
              }
            }
            soft_sync();
            if (sidx < n_pad) {
              const int i = i0 + (sidx >> (__ffs(p.G) - 1));  // block row of query column sidx
              const int krow = sg.L + i - kt;                  // its own key's place in the tile
              const bool seen = sidx < m_valid && sg.L + i >= vstart;
              mnew[sidx] = seen ? reinterpret_cast<const float*>(sm + S::P_OFF)[krow * 64 + sidx] * c : -CUDART_INF_F;
            }
          }
          soft_sync();
          mpar ^= 1;
          mref = mref_buf + mpar * S::RS;
        }
        // ---- pass 0: score - reference; does any exceed 2^60? -----------------
        bool over = false;
        if (!over) {
          // (independent maxima per piece: a single running flag would chain every element)
          float worst[MAXP];
#pragma unroll
          for (int j = 0; j < MAXP; ++j) {
            worst[j] = -CUDART_INF_F;
            if (j < np) {
              const float4 m0 = reinterpret_cast<const float4*>(mref + col0 + j * 8)[0];
              const float4 m1 = reinterpret_cast<const float4*>(mref + col0 + j * 8)[1];
              const float mm[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
#pragma unroll
              for (int e = 0; e < 8; ++e) sv[j][e] = fmaf(sv[j][e], c, -mm[e]);
              if (!masked) {
                worst[j] = fmaxf(fmaxf(fmaxf(sv[j][0], sv[j][1]), fmaxf(sv[j][2], sv[j][3])),
                                 fmaxf(fmaxf(sv[j][4], sv[j][5]), fmaxf(sv[j][6], sv[j][7])));
              } else {
                const uint32_t vb = (uint32_t)(vis >> (j * 8)) & 0xFFu;
#pragma unroll
                for (int e = 0; e < 8; ++e)
                  worst[j] = fmaxf(worst[j], ((vb >> e) & 1u) ? sv[j][e] : -CUDART_INF_F);
              }
            }
          }
          float w = worst[0];
#pragma unroll
          for (int j = 1; j < MAXP; ++j) w = fmaxf(w, worst[j]);
          over = !(w <= OVER_THRESHOLD);                    // also true for NaN
        }
        if (soft_any(over)) {
          // ---- re-reference: per query row maximum over the 128 keys of this tile
#pragma unroll
          for (int j = 0; j < MAXP; ++j)
            if (j < np) piece_key_max(ts + j * 8, (uint32_t)(vis >> (j * 8)) & 0xFFu, xq + quarter * S::RS + col0 + j * 8);
          soft_sync();
          // PV of the previous tile must be done before O^T is rescaled
          if (!first) {
            ok &= mbar_wait(BAR(B_PVDONE + ((gt - 1) & 1)), ((gt - 1) >> 1) & 1, abort_flag, p.err, 10);
            tc_fence_after();
          }
          float* mnew = mref_buf + (mpar ^ 1) * S::RS;
#pragma unroll
          for (int j = 0; j < MAXP; ++j) {
            if (j < np) {
              const int q0 = col0 + j * 8;
              // fq is written and read back by the same thread (its peers write identical values)
              piece_new_reference(xq + q0, S::RS, mref + q0, mnew + q0, fq + q0, c, first);
              __syncwarp();
              if (!first) {
#pragma unroll
                for (int e = 0; e < 8; ++e) lsum[j][e] *= fq[q0 + e];
                piece_rescale(TM_O + lane_addr + q0, fq + q0);
                piece_rescale(TM_O + lane_addr + 64 + q0, fq + q0);
              }
              // scores again, now against the new reference
              uint32_t sr[8];
              tmem_ld8(ts + j * 8, sr);
              tmem_wait_ld();
#pragma unroll
              for (int e = 0; e < 8; ++e) sv[j][e] = fmaf(__uint_as_float(sr[e]), c, -mnew[q0 + e]);
            }
          }
          mpar ^= 1;
          mref = mref_buf + mpar * S::RS;
          soft_sync();                                      // new references visible to every thread
        }
        // the P buffer is free once the PV product that last read it has finished
        {
          const uint32_t prev = gt - S::P_BUFS;             // tile that used this P buffer before
          if (gt >= (uint32_t)S::P_BUFS)
            ok &= mbar_wait(BAR(B_PVDONE + (prev & 1)), (prev >> 1) & 1, abort_flag, p.err, 11);
        }
        const uint32_t pbuf = prow + (gt % S::P_BUFS) * (2 * S::P_PART);
        // ---- pass 1: P = exp2(score - reference) as P_hi + P_lo (two bf16 terms:
        // bf16 alone leaves an output error near 1e-2 of the output RMS)
#pragma unroll
        for (int j = 0; j < MAXP; ++j) {
          if (j < np) {
            uint32_t hi[4], lw[4];
#pragma unroll
            for (int e2 = 0; e2 < 4; ++e2) {
              float p0 = fast_exp2(sv[j][2 * e2]), p1 = fast_exp2(sv[j][2 * e2 + 1]);
              if (masked) {
                // a row without any visible key so far has reference -inf and only
                // invisible entries: the select keeps those at zero
                p0 = ((vis >> (j * 8 + 2 * e2)) & 1ull) ? p0 : 0.f;
                p1 = ((vis >> (j * 8 + 2 * e2 + 1)) & 1ull) ? p1 : 0.f;
              }
              lsum[j][2 * e2] += p0;
              lsum[j][2 * e2 + 1] += p1;
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);        // .x = lower query row
              const float2 hf = __bfloat1622float2(h2);
              const __nv_bfloat162 l2 = __floats2bfloat162_rn(p0 - hf.x, p1 - hf.y);
              hi[e2] = *reinterpret_cast<const uint32_t*>(&h2);
              lw[e2] = *reinterpret_cast<const uint32_t*>(&l2);
            }
            // P^T rows are keys; a row holds 64 query rows as eight 16-byte pieces,
            // piece j stored at j ^ (key & 7) (128-byte swizzle)
            const int q0 = col0 + j * 8;
            const uint32_t dst = pbuf + (uint32_t)(q0 >> 6) * (TILE_N * 128) + ((((uint32_t)(q0 & 63) >> 3) ^ swz) << 4);
            st_shared_v4(dst, hi[0], hi[1], hi[2], hi[3]);
            st_shared_v4(dst + S::P_PART, lw[0], lw[1], lw[2], lw[3]);
          }
        }
        if (PAGED && kt + TILE_N > n_keys) {
          // Paged cache, last tile: the page's rows past the last key may hold anything, and 0 * NaN
          // would reach O^T.  Once the V tile has landed, the thread of such a row clears it (a row
          // is 128 contiguous bytes per 64-wide half of d, whatever the swizzle inside them).
          const uint32_t vs = gt % S::V_STAGES;
          ok &= mbar_wait(BAR(B_VFULL + vs), (gt / S::V_STAGES) & 1, abort_flag, p.err, 17);
          if (key >= n_keys) {
            for (int hf = half; hf < S::HALVES; hf += 2) {
              const uint32_t vrow = sm_base + S::V_OFF + vs * S::TILE_BYTES + hf * (TILE_N * 128) + kl * 128;
#pragma unroll
              for (int i = 0; i < 8; ++i) st_shared_v4(vrow + i * 16, 0u, 0u, 0u, 0u);
            }
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // P (and a cleared V row) is read by the tensor core
        tc_fence_before();
        mbar_arrive(BAR(B_PREADY + buf));
        if (sidx == 0) { if (gt == 0) TL(6); TL(9); }
      }
      // ---- end of share: final output or partial ---------------------------
      // Row sums first, while the last O^T product still runs.  Every thread holds
      // its key's share of up to 32 rows; a halving butterfly over the warp leaves
      // lane r with the sum over the warp's 32 keys for row col0 + r
      // (with two 64-row blocks: two such folds, rows col0 + r and col0 + 32 + r)
#pragma unroll
      for (int f0 = 0; f0 < MAXP * 8; f0 += 32) {
        float red[32];
#pragma unroll
        for (int x = 0; x < 32; ++x) {
          const int j = (f0 + x) >> 3, e = (f0 + x) & 7;     // piece and element, compile-time after unrolling
          red[x] = (j < MAXP && j < np) ? lsum[j < MAXP ? j : 0][e] : 0.f;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const bool up = (lane & o) != 0;
#pragma unroll
          for (int i = 0; i < o; ++i) {
            const float send = up ? red[i] : red[i + o];
            const float keep = up ? red[i + o] : red[i];
            red[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, o);
          }
        }
        if (f0 + lane < ncol) xq[quarter * S::RS + col0 + f0 + lane] = red[0];
      }
      soft_sync();
      float* rcp = mref_buf + (mpar ^ 1) * S::RS;            // the idle copy of the references
      if (sidx < n_pad) {
        const float v = (xq[sidx] + xq[S::RS + sidx]) + (xq[2 * S::RS + sidx] + xq[3 * S::RS + sidx]);
        fq[sidx] = v;                                        // row sums and their reciprocals
        rcp[sidx] = 1.f / v;
      }
      ok &= mbar_wait(BAR(B_PVDONE + ((gt - 1) & 1)), ((gt - 1) >> 1) & 1, abort_flag, p.err, 12);
      tc_fence_after();
      soft_sync();
      if (sidx == 0) TL(10);
      const bool whole = sg.n == sg.T;
      const int item = sg.b * p.H_kv + sg.h;
      float* pslot = p.part + ((size_t)sg.slot * p.n_mblocks + mb) * (ROWS * (DH + 2));
      if (sidx == 0 && ok) {
        // how this (sequence, head) was cut, read by attn_merge_kernel (every group of
        // the cut writes the same pair)
        // {first partial slot, number of partials}
        int2 d = make_int2(sg.slot, 1);
        if (sg.dfirst >= 0) {
          d = make_int2(sg.dfirst, sg.dn);
        } else if (!whole) {
          const long long W = prefix[p.B];
          const long long NG = W < p.n_groups ? W : p.n_groups;
          const long long f0 = (long long)prefix[sg.b] + (long long)sg.h * (sg.T + SHARE_COST);
          const int g0 = group_of(f0 + SHARE_COST, W, NG);  // group of the first tile
          d.x = item + g0;
          d.y = group_of(f0 + SHARE_COST + sg.T - 1, W, NG) - g0 + 1;
        }
        p.desc[(size_t)item * p.n_mblocks + mb] = d;
        if (!whole && sg.tile_at(sg.n - 1) == sg.T - 1) own = item;   // the piece with the pair's last tile; at most one per block
      }
      if (sidx < m_valid && ok) {                           // per-row scalars
        const int q = sidx;
        if (whole) {
          if (p.lse) {
            const int i = i0 + q / p.G, hq = sg.h * p.G + q % p.G;
            p.lse[((size_t)sg.b * p.H_q + hq) * p.n_q + i] = (mref[q] + log2f(fq[q])) * 0.6931471805599453f;
          }
        } else {
          pslot[ROWS * DH + q] = mref[q];
          pslot[ROWS * DH + ROWS + q] = fq[q];
        }
      }
      // O^T: lane = head-dim index, column = query row.  A warp writes 32
      // consecutive floats of one output row per store.
      const bool d_ok = kl < DH && ok;                      // lanes 64..127 repeat 0..63 when head_dim is 64
      const int gsh = __ffs(p.G) - 1;
      const bool out_f32 = p.out_dtype == SPACE_DTYPE_F32;
      // element (block row i0, head h*G, dim kl) of this sequence; one block row further = H_q*DH
      const size_t out_base = (((size_t)sg.b * p.n_q + i0) * p.H_q + (size_t)sg.h * p.G) * DH + kl;
      const size_t out_row = (size_t)p.H_q * DH;
#pragma unroll 2
      for (int j = 0; j < np; ++j) {
        uint32_t o[8], o2[8];
        const int q0 = col0 + j * 8;
        tmem_ld8(TM_O + lane_addr + q0, o);
        tmem_ld8(TM_O + lane_addr + 64 + q0, o2);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 8; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) + __uint_as_float(o2[e]));
        if (whole) {
          // query row q of the block is head q mod G of block row q / G (G is a power of two)
          const float4 r0 = reinterpret_cast<const float4*>(rcp + q0)[0], r1 = reinterpret_cast<const float4*>(rcp + q0)[1];
          const float rr[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
          size_t off[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const int q = q0 + e;
            off[e] = out_base + (size_t)(q >> gsh) * out_row + (size_t)(q & (p.G - 1)) * DH;
          }
          if (out_f32) {
#pragma unroll
            for (int e = 0; e < 8; ++e)
              if (q0 + e < m_valid && d_ok) reinterpret_cast<float*>(p.out)[off[e]] = __uint_as_float(o[e]) * rr[e];
          } else {
#pragma unroll
            for (int e = 0; e < 8; ++e)
              if (q0 + e < m_valid && d_ok)
                reinterpret_cast<__nv_bfloat16*>(p.out)[off[e]] = __float2bfloat16_rn(__uint_as_float(o[e]) * rr[e]);
          }
        } else {
          float* dst = pslot + (size_t)q0 * DH + kl;
#pragma unroll
          for (int e = 0; e < 8; ++e)
            if (q0 + e < m_valid && d_ok) dst[e * DH] = __uint_as_float(o[e]);
        }
      }
      tc_fence_before();
      soft_sync();                                          // scratch, fq and mref are reused by the next share
      if (sidx == 0) TL(11);
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
  if (threadIdx.x == 32) TL(13);                          // after the TMEM release
}

// Combine the partials of every (sequence, kv head, query-row block) that was
// cut over several groups: one thread per 16 output bytes, all loads of a
// thread independent, running maximum / denominator / accumulator in one pass.
// grid = (B*H_kv*n_mblocks, ceil(rows*DH/4 / 128)), 128 threads.
template <int DH>
__global__ void __launch_bounds__(128) attn_merge_kernel(const AttnParams p) {
  TLM(0);
  pdl_launch_dependents();
  pdl_wait();
  TLM(1);
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
  TLM(2);
  if (n <= 1) return;                                       // written directly by the main kernel
  const int i0 = mb * p.rows_per_mb;
  const int m_valid = min(p.rows_per_mb, p.n_q - i0) * p.G;
  const int idx = blockIdx.y * 128 + threadIdx.x;
  if (idx >= m_valid * C4) return;
  const int r = idx / C4, c4 = idx % C4;
  const size_t slot_floats = (size_t)ROWS * (DH + 2);
  const float* ps = p.part + ((size_t)d.x * p.n_mblocks + mb) * slot_floats;
  const size_t gstride = (size_t)p.n_mblocks * slot_floats;
  float mx = -CUDART_INF_F, den = 0.f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  // batches of eight partials: all loads of a batch are issued before any is used
  for (int x0 = 0; x0 < n; x0 += 8) {
    float ms[8], ls[8];
    float4 ov[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (x0 + j < n) {
        const float* pj = ps + (size_t)(x0 + j) * gstride;
        ms[j] = __ldcg(pj + ROWS * DH + r);
        ls[j] = __ldcg(pj + ROWS * DH + ROWS + r);
        ov[j] = __ldcg(reinterpret_cast<const float4*>(pj + (size_t)r * DH) + c4);
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (x0 + j < n) {
        const float mn = fmaxf(mx, ms[j]);
        if (mn > -CUDART_INF_F) {
          const float e0 = fast_exp2(mx - mn), e1 = fast_exp2(ms[j] - mn);
          den = den * e0 + ls[j] * e1;
          acc.x = acc.x * e0 + ov[j].x * e1; acc.y = acc.y * e0 + ov[j].y * e1;
          acc.z = acc.z * e0 + ov[j].z * e1; acc.w = acc.w * e0 + ov[j].w * e1;
        }
        mx = mn;
      }
    }
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
  TLM(3);
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
  const int max_rows = 112 / G;                             // (block row, head) pairs per thread block: at most 112
  pl->n_mblocks = (n_q + max_rows - 1) / max_rows;
  pl->rows_per_mblock = (n_q + pl->n_mblocks - 1) / pl->n_mblocks;
  int groups = sm_count / pl->n_mblocks;
  if (groups < 1) groups = 1;
  pl->n_ctas = groups * pl->n_mblocks;
}

template <int DH>
size_t smem_bytes(int max_batch) {
  return Smem<DH>::TABLE_OFF + (size_t)(2 * max_batch + 1) * sizeof(int);
}

template <int DH, bool PAGED>
cudaError_t launch_main(const AttnParams& p, int n_ctas, int max_batch, cudaStream_t st) {
  const size_t sm = smem_bytes<DH>(max_batch);
  // the shared-memory limit of the kernel is raised once per device (to the most any batch needs)
  static unsigned long long done_mask = 0;                 // (one per instantiation)
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 64 || !((done_mask >> dev) & 1ull)) {
    cudaFuncSetAttribute(attn_tc_kernel<DH, PAGED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         (int)smem_bytes<DH>(128));
    if (dev < 64) done_mask |= 1ull << dev;
  }
  return launch_pdl(attn_tc_kernel<DH, PAGED>, dim3(n_ctas), dim3(THREADS), sm, st, p, max_batch);
}

}  // namespace

size_t attn_tensor_partial_floats(const space_config* cfg, int sm_count, size_t* slots_out) {
  AttnPlanHost pl;
  plan(cfg, sm_count, cfg->k_max, &pl);
  // the largest slot index is (B*H_kv - 1) + (groups - 1), times the query-row blocks
  size_t worst_mb = 1;
  for (int k = 1; k <= cfg->k_max; ++k) {
    AttnPlanHost q; plan(cfg, sm_count, k, &q);
    if ((size_t)q.n_mblocks > worst_mb) worst_mb = q.n_mblocks;
  }
  const size_t slots = ((size_t)cfg->max_batch * cfg->n_kv_heads + sm_count) * worst_mb;
  if (slots_out) *slots_out = slots;
  return slots * (size_t)ROWS * (cfg->head_dim + 2);
}

#ifdef SPACE_TIMELINE
extern "C" int space_debug_timeline_read(unsigned long long* host_dst, int n_blocks) {
  return cuda_ok(cudaMemcpyFromSymbol(host_dst, g_timeline, sizeof(unsigned long long) * TL_POINTS * n_blocks));
}
extern "C" int space_debug_timeline_read_merge(unsigned long long* host_dst, int n_blocks) {
  return cuda_ok(cudaMemcpyFromSymbol(host_dst, g_timeline_merge, sizeof(unsigned long long) * 4 * n_blocks));
}
#endif

int launch_attn_tensor(space_ctx* ctx, const space_attn_args* a, const uint64_t* mask_rows,
                       cudaStream_t st) {
  const space_config& cfg = ctx->cfg;
  const int DH = cfg.head_dim;
  AttnPlanHost pl;
  plan(&cfg, ctx->sm_count, a->k, &pl);
  // Query blocks wider than 64 rows per kv head are better served by the kernel
  // with the query rows on the M extent (measured), which can also be asked for.
  if (a->impl == SPACE_ATTN_TENSOR_ROWS ||
      ((pl.rows_per_mblock * (cfg.n_q_heads / cfg.n_kv_heads) + 15) / 16) * 16 > 64)
    return launch_attn_rows(ctx, a, mask_rows, st);
  AttnParams p;
  memset(&p, 0, sizeof(p));
  p.B = a->batch; p.n_q = (a->k + 1) * (a->k + 1);
  p.H_q = cfg.n_q_heads; p.H_kv = cfg.n_kv_heads; p.G = p.H_q / p.H_kv;
  p.n_mblocks = pl.n_mblocks; p.rows_per_mb = pl.rows_per_mblock;
  p.n_groups = pl.n_ctas / pl.n_mblocks;
  p.n_pad = ((pl.rows_per_mblock * p.G + 15) / 16) * 16;
  p.out_dtype = a->out_dtype;
  p.s_cap = a->page_table ? (int64_t)a->pages_per_seq * SPACE_PAGE_SIZE : cfg.s_cap;
  p.page_table = a->page_table; p.pages_per_seq = a->pages_per_seq; p.n_pages = a->n_pages;
  p.scale_log2 = a->scale * 1.4426950408889634f;
  p.kv_len = a->kv_len; p.out = a->out; p.lse = a->lse; p.status = a->status;
  p.part = ctx->attn_part; p.err = ctx->counters + 3 * cfg.max_batch;
  p.desc = reinterpret_cast<int2*>(ctx->merge_cnt);
  p.owner = ctx->merge_cnt + (size_t)cfg.max_batch * cfg.n_kv_heads * 8 * 2;
  p.merge_by_owner = (a->batch * p.H_kv * p.n_mblocks > pl.n_ctas) ? 1 : 0;
  p.spec = (a->batch == 1 && p.H_kv <= p.n_groups) ? 1 : 0;
  if (p.n_mblocks > 2) return SPACE_E_UNSUPPORTED;         // (cannot happen: at most 64 block rows, at least 32 per block)
  if (ctx->visq_k != a->k || ctx->visq_variant != a->mask_variant) {
    memset(ctx->visq, 0, sizeof(ctx->visq));
    for (int m = 0; m < p.n_mblocks; ++m) {
      const int i0 = m * p.rows_per_mb;
      const int rows = (p.n_q - i0 < p.rows_per_mb ? p.n_q - i0 : p.rows_per_mb);
      for (int j = 0; j < SPACE_MAX_ROWS; ++j) {
        uint64_t v = 0;
        for (int q = 0; q < rows * p.G; ++q) v |= ((mask_rows[i0 + q / p.G] >> j) & 1ull) << q;
        ctx->visq[m][j] = v;
      }
    }
    ctx->visq_k = a->k; ctx->visq_variant = a->mask_variant;
  }
  memcpy(p.visq, ctx->visq, sizeof(p.visq));

  // TMA descriptors, rebuilt only when a base pointer or a stride changes
  const int64_t key[8] = {a->kv_stride_b, a->kv_stride_h, a->kv_stride_s, a->batch, p.n_q, p.n_pad,
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
    const cuuint32_t qb[4] = {64, (cuuint32_t)p.G, (cuuint32_t)(p.n_pad / p.G), 1};
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
  {
    ProfScope ps(ctx, SPACE_K_ATTN, st);
    if (a->page_table) {
      if (DH == 128) launch_main<128, true>(p, pl.n_ctas, cfg.max_batch, st);
      else launch_main<64, true>(p, pl.n_ctas, cfg.max_batch, st);
    } else {
      if (DH == 128) launch_main<128, false>(p, pl.n_ctas, cfg.max_batch, st);
      else launch_main<64, false>(p, pl.n_ctas, cfg.max_batch, st);
    }
  }
  {
    ProfScope ps(ctx, SPACE_K_MERGE, st);
    if (DH == 128) launch_pdl(attn_merge_kernel<128>, mgrid, dim3(128), 0, st, p);
    else launch_pdl(attn_merge_kernel<64>, mgrid, dim3(128), 0, st, p);
  }
  ctx->launches += 2;
  return cuda_ok(cudaGetLastError());
}
