// Internal declarations shared by the translation units of libspace.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "../../include/space.h"
#include <cstring>

#define SPACE_VERIFY_MAX_CHUNKS 64
#define SPACE_VERIFY_THREADS 256
#define SPACE_FUSED_MAX_CHUNKS 16

// ---- Philox4x32-10 (Salmon et al., SC'11) ---------------------------------
struct Philox4 { uint32_t x, y, z, w; };

__host__ __device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2,
                                                          uint32_t c3, uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    c1 = (uint32_t)p1;
    c3 = (uint32_t)p0;
    c0 = n0;
    c2 = n2;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return Philox4{c0, c1, c2, c3};
}

// 32-bit word -> uniform in (0,1), exactly representable in binary32.
// ((w >> 9) + 1/2) 2^-23, built without an integer-to-float conversion: the 23 bits
// become the mantissa of a float in [1, 2), and subtracting 1 - 2^-24 (the largest
// float below 1) leaves (2m + 1) 2^-24 exactly.
__host__ __device__ __forceinline__ float uniform_open(uint32_t w) {
  const uint32_t bits = 0x3F800000u | (w >> 9);
  float f;
#ifdef __CUDA_ARCH__
  f = __uint_as_float(bits);
#else
  memcpy(&f, &bits, sizeof(f));
#endif
  return f - 0.99999994f;
}

enum { PURPOSE_ACCEPT = 0, PURPOSE_TOKEN = 1, PURPOSE_DRAFT = 2 };

// Gumbel noise in units of log 2:  -log2(-log2 u)  for u = (m + 1/2) 2^-23.
// arg-max_x (z_x/T - log(-log u_x)) = arg-max_x (z_x*log2(e)/T - log2(-log2 u_x)):
// the two scores differ by the factor log 2 and a constant, so the hardware
// base-2 logarithm serves without rescaling.  Near u = 1 the inner logarithm is
// taken from its series in d = 1 - u (exact in binary32); the error of the result
// stays below 3e-5, inside the 1e-4 band within which two scores count as tied.
__device__ __forceinline__ float fast_log2(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float gumbel2_from_uniform(float u) {
  const float d = 1.0f - u;
  const float t = (d < 0.0078125f) ? d * (1.0f + d * (0.5f + d * 0.33333334f)) * 1.4426950408889634f
                                   : -fast_log2(u);
  return -fast_log2(t);
}


// ---- context ---------------------------------------------------------------
struct VerifyPartial { float m, s, gs; int idx, gidx, pad0, pad1, pad2; };   // 32 bytes
struct VerifyRow     { float m, s; int idx, pad; };

struct AttnPlanHost {
  int n_ctas;         // persistent grid size
  int n_mblocks;      // query-row blocks per (sequence, kv head)
  int rows_per_mblock;// block rows (i) per query-row block
};

struct space_ctx {
  space_config cfg;
  int sm_count;
  int64_t launches;
  // one allocation, carved up
  char* ws;
  size_t ws_bytes;
  float* attn_part;        // split partials
  size_t attn_part_slots;
  int* counters;           // [4][max_batch] self-resetting arrival counters
  int* merge_cnt;          // attention split arrivals, one per (sequence, kv head, row block)
  VerifyPartial* vpart;    // [max_batch][k_max+2][SPACE_VERIFY_MAX_CHUNKS]
  VerifyRow* vrow;         // [max_batch][k_max+1]
  VerifyPartial* vfused;   // [max_batch][SPACE_MAX_ROWS][16] single-launch greedy path
  char* vtopk;             // filtered sampling: top-k lists per (sequence, row, chunk)
  int32_t* scratch_status; // [max_batch] used when the caller passes no status array
  char* lm_part;           // output-projection statistics [256 block rows][sm_count] x 16 bytes
  int* lm_counter;         // {arrival counter, first timeout site}
  // staging for space_step_host
  char* stage;
  char* host_small;        // pinned host mirror of the staging area's small per-sequence arrays (host_staging only)
  cudaStream_t aux_stream; // space_step_host: second stream, so that the logits upload and the download of the
  cudaEvent_t aux_ev[4];   //   attention output overlap the kernels (host_staging only)
  size_t stage_bytes;
  // per-kernel event timing (space_profile_*)
  int prof_on;
  int prof_n[SPACE_K_COUNT];
  cudaEvent_t* prof_ev[SPACE_K_COUNT];   // [2 * SPACE_PROFILE_MAX_STEPS] start/stop pairs, lazily created
  // cached block layout (Eq. 5 mask rows) and the attention kernel's visibility words, per (k, mask variant)
  int lay_k, lay_variant;                // lay_k = 0: nothing cached
  uint64_t lay_mask[SPACE_MAX_ROWS];
  int visq_k, visq_variant;
  uint64_t visq[2][SPACE_MAX_ROWS];
  // cached TMA descriptors
  const void* tm_q_ptr; const void* tm_k_ptr; const void* tm_v_ptr;
  int64_t tm_key[8];
  alignas(64) unsigned char tm_q[128];
  alignas(64) unsigned char tm_k[128];
  alignas(64) unsigned char tm_v[128];
};

// ---- KV commit: shared by kv_commit_kernel and the verify kernels that carry the commit ----
// Rows L + g(k+1) -> L + g, g = 1..i*, of K and V for every kv head (16-byte pieces).
struct CommitParams {
  int B, k, H_kv, d, blocks_per_seq, in_place;
  int64_t s_cap;
  __nv_bfloat16* kc; __nv_bfloat16* vc;
  int64_t sb, sh, ss;
  const int32_t* n_accept; const int32_t* kv_len;
  int32_t* kv_len_out; int32_t* src; int32_t* dst; int32_t* status;
  int* counter;
  const int32_t* page_table; int pages_per_seq, n_pages;   // paged cache (page_table != nullptr): kc / vc are page pools
};

// Row s of sequence b, head h, of a cache that is contiguous (page_table == nullptr) or paged:
// offset in elements from the cache base, or -1 for a page-table entry outside the pool.
__device__ __forceinline__ int64_t kv_row_offset(const int32_t* page_table, int pages_per_seq, int n_pages,
                                                 int64_t sb, int64_t sh, int64_t ss, int b, int h, int s) {
  if (!page_table) return (int64_t)b * sb + (int64_t)h * sh + (int64_t)s * ss;
  const int pg = page_table[(int64_t)b * pages_per_seq + s / SPACE_PAGE_SIZE];
  if (pg < 0 || pg >= n_pages) return -1;
  return (int64_t)pg * sb + (int64_t)h * sh + (int64_t)(s % SPACE_PAGE_SIZE) * ss;
}

__device__ __forceinline__ bool commit_fits(const CommitParams& p, int L) {
  return L >= 0 && (int64_t)L + (int64_t)(p.k + 1) * (p.k + 1) <= p.s_cap;
}

// Slice `part` of `nparts` of sequence b's move, by `nthreads` threads (this one is `tid`).
// All loads of a batch are issued before its stores.
template <bool PAGED>
__device__ __forceinline__ void commit_rows_impl(const CommitParams& p, int b, int L, int i_star, int part, int nparts,
                                                 int tid, int nthreads) {
  const int k1 = p.k + 1;
  const int vec_per_row = p.d / 8;                      // 16-byte pieces per row
  const int total = i_star * p.H_kv * 2 * vec_per_row;
  const int stride = nparts * nthreads;
  constexpr int U = 8;
  for (int t0 = part * nthreads + tid; t0 < total; t0 += U * stride) {
    uint4 val[U];
    uint4* dd[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int t = t0 + u * stride;
      dd[u] = nullptr;
      if (t < total) {
        int r = t;
        const int v = r % vec_per_row; r /= vec_per_row;
        const int which = r % 2;       r /= 2;
        const int h = r % p.H_kv;      r /= p.H_kv;
        const int g = r + 1;                            // accepted candidate g = 1..i*
        if (!PAGED) {
          __nv_bfloat16* base = (which ? p.vc : p.kc) + (int64_t)b * p.sb + (int64_t)h * p.sh;
          val[u] = *(reinterpret_cast<const uint4*>(base + (int64_t)(L + g * k1) * p.ss) + v);
          dd[u] = reinterpret_cast<uint4*>(base + (int64_t)(L + g) * p.ss) + v;
        } else {
          __nv_bfloat16* base = which ? p.vc : p.kc;
          const int64_t so = kv_row_offset(p.page_table, p.pages_per_seq, p.n_pages, p.sb, p.sh, p.ss, b, h, L + g * k1);
          const int64_t dof = kv_row_offset(p.page_table, p.pages_per_seq, p.n_pages, p.sb, p.sh, p.ss, b, h, L + g);
          if (so >= 0 && dof >= 0) {
            val[u] = *(reinterpret_cast<const uint4*>(base + so) + v);
            dd[u] = reinterpret_cast<uint4*>(base + dof) + v;
          } else if (p.status && v == 0 && which == 0 && h == 0) {
            atomicOr(p.status + b, SPACE_ST_BAD_PAGE);        // the row stays where it is
          }
        }
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u)
      if (dd[u]) *dd[u] = val[u];
  }
}

// Contiguous cache only: the form the verify kernels carry (it sits in their critical path; with a
// paged cache space_verify_commit runs the commit kernel after them instead).
__device__ __forceinline__ void commit_rows(const CommitParams& p, int b, int L, int i_star, int part, int nparts,
                                            int tid, int nthreads) {
  commit_rows_impl<false>(p, b, L, i_star, part, nparts, tid, nthreads);
}
// Either cache form (the commit kernel).
__device__ __forceinline__ void commit_rows_any(const CommitParams& p, int b, int L, int i_star, int part, int nparts,
                                                int tid, int nthreads) {
  if (p.page_table) commit_rows_impl<true>(p, b, L, i_star, part, nparts, tid, nthreads);
  else commit_rows_impl<false>(p, b, L, i_star, part, nparts, tid, nthreads);
}

// New length and index tables of sequence b (one thread).
__device__ __forceinline__ void commit_tables(const CommitParams& p, int b, int L, int i_star, bool fits) {
  const int k1 = p.k + 1;
  if (!fits) {
    if (p.status) atomicOr(p.status + b, SPACE_ST_CAPACITY);
    i_star = -1;                                        // nothing committed, length unchanged
  }
  if (p.kv_len_out) p.kv_len_out[b] = L + i_star + 1;
  for (int g = 0; g < k1; ++g) {
    if (p.src) p.src[b * k1 + g] = (g <= i_star) ? L + g * k1 : -1;
    if (p.dst) p.dst[b * k1 + g] = (g <= i_star) ? L + g : -1;
  }
}

// ---- per-stage launchers (defined next to their kernels) -------------------
// cm != nullptr: the verify kernels also carry out the commit described by cm (one launch less)
int launch_verify(space_ctx* ctx, const space_verify_args* a, const space_commit_args* cm, cudaStream_t st);
int launch_verify_filtered(space_ctx* ctx, const space_verify_args* a, cudaStream_t st);
size_t verify_filter_scratch_bytes(int max_batch, int k_max);
void fill_commit_params(const space_ctx* ctx, const space_commit_args* a, CommitParams* p);
int launch_verify_noalloc(const space_verify_args* a, cudaStream_t st);
int launch_commit(space_ctx* ctx, const space_commit_args* a, cudaStream_t st);
int launch_lmhead_verify(space_ctx* ctx, const space_lmhead_args* a, cudaStream_t st);
size_t lmhead_partial_bytes(int sm_count);
int launch_attn_simt(space_ctx* ctx, const space_attn_args* a, const uint64_t* mask_rows,
                     cudaStream_t st);
int launch_attn_tensor(space_ctx* ctx, const space_attn_args* a, const uint64_t* mask_rows,
                       cudaStream_t st);
int launch_attn_rows(space_ctx* ctx, const space_attn_args* a, const uint64_t* mask_rows, cudaStream_t st);
size_t attn_tensor_partial_floats(const space_config* cfg, int sm_count, size_t* slots);
int launch_philox_debug(uint64_t seed, int64_t n, const uint32_t* c0, const uint32_t* c1,
                        const uint32_t* c2, const uint32_t* c3, uint32_t* out, cudaStream_t st);

// Event pair around one kernel launch when profiling is on.
struct ProfScope {
  space_ctx* ctx; int which; cudaStream_t st; int slot;
  ProfScope(space_ctx* c, int w, cudaStream_t s) : ctx(c), which(w), st(s), slot(-1) {
    if (!c->prof_on || !c->prof_ev[w] || c->prof_n[w] >= SPACE_PROFILE_MAX_STEPS) return;
    slot = c->prof_n[w];
    cudaEventRecord(c->prof_ev[w][2 * slot], st);
  }
  ~ProfScope() {
    if (slot < 0) return;
    cudaEventRecord(ctx->prof_ev[which][2 * slot + 1], st);
    ctx->prof_n[which] = slot + 1;
  }
};

// Programmatic dependent launch: the kernel may be scheduled while the previous
// kernel of the stream is still draining; every kernel calls pdl_wait() before
// it touches global memory, which blocks until the previous kernel has finished
// and its writes are visible.  Both are no-ops without the launch attribute.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                     cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

static inline int cuda_ok(cudaError_t e) { return e == cudaSuccess ? SPACE_OK : SPACE_E_CUDA; }
