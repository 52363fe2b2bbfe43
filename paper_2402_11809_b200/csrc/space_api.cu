// Host side of libspace: context, argument validation, block layout, and the
// exported entry points declared in include/space.h.
#include "common.cuh"
#include "tc_common.cuh"
#include <cstdlib>
#include <cstring>
#include <new>

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool config_ok(const space_config* c) {
  if (!c) return false;
  if (c->max_batch < 1 || c->max_batch > 128) return false;
  if (c->n_q_heads < 1 || c->n_kv_heads < 1 || c->n_q_heads % c->n_kv_heads) return false;
  if (c->k_max < 1 || c->k_max > SPACE_MAX_K) return false;
  if (c->s_cap < (int64_t)(c->k_max + 1) * (c->k_max + 1) || c->s_cap > (1ll << 30)) return false;
  if (c->vocab < 1) return false;
  return true;
}

int config_supported(const space_config* c) {
  const int G = c->n_q_heads / c->n_kv_heads;
  if (c->head_dim != 64 && c->head_dim != 128) return SPACE_E_UNSUPPORTED;
  if (G != 1 && G != 2 && G != 4 && G != 8 && G != 16) return SPACE_E_UNSUPPORTED;
  return SPACE_OK;
}

struct Carve {
  size_t attn_part, counters, merge_cnt, vtopk, vpart, vfused, vrow, status, lm_part, lm_counter, stage, total;
  size_t part_slots;
  // staging sub-offsets (relative to stage)
  size_t st_q, st_k, st_v, st_logits, st_small;
};

Carve carve(const space_config* c, int sm_count) {
  Carve v{};
  size_t off = 0;
  v.attn_part = off;
  off += align_up(attn_tensor_partial_floats(c, sm_count, &v.part_slots) * sizeof(float), 256);
  v.counters = off; off += align_up((size_t)(3 * c->max_batch + 4) * sizeof(int), 256);
  v.merge_cnt = off;
  // up to 8 row blocks, one {first, count} pair each; then one word per thread block of the attention grid
  off += align_up((size_t)c->max_batch * c->n_kv_heads * 8 * sizeof(int2) + (size_t)(sm_count + 8) * sizeof(int), 256);
  v.vtopk = off; off += align_up(verify_filter_scratch_bytes(c->max_batch, c->k_max), 256);
  v.vpart = off;
  off += align_up((size_t)c->max_batch * (c->k_max + 2) * SPACE_VERIFY_MAX_CHUNKS * sizeof(VerifyPartial), 256);
  static_assert(SPACE_FUSED_MAX_CHUNKS <= 16, "the single-launch verify reduces a row's chunks with 16 lanes");
  v.vfused = off; off += align_up((size_t)c->max_batch * SPACE_MAX_ROWS * SPACE_FUSED_MAX_CHUNKS * sizeof(VerifyPartial), 256);
  v.vrow = off; off += align_up((size_t)c->max_batch * (c->k_max + 1) * sizeof(VerifyRow), 256);
  v.status = off; off += align_up((size_t)c->max_batch * sizeof(int32_t), 256);
  v.lm_part = off; off += align_up(lmhead_partial_bytes(sm_count), 256);
  // counter, error word; one arg-max key per block row; one candidate logit per block row
  v.lm_counter = off; off += 256 + 256 * sizeof(unsigned long long) + 256 * sizeof(float);
  v.stage = off;
  if (c->host_staging) {
    const size_t n_q = (size_t)(c->k_max + 1) * (c->k_max + 1);
    size_t s = 0;
    v.st_q = s; s += align_up((size_t)c->max_batch * n_q * c->n_q_heads * c->head_dim * 2, 256);
    v.st_k = s; s += align_up((size_t)c->max_batch * c->n_kv_heads * c->s_cap * c->head_dim * 2, 256);
    v.st_v = s; s += align_up((size_t)c->max_batch * c->n_kv_heads * c->s_cap * c->head_dim * 2, 256);
    v.st_logits = s; s += align_up((size_t)c->max_batch * n_q * c->vocab * 4, 256);
    v.st_small = s;
    // out (f32) + a handful of small per-sequence arrays
    s += align_up((size_t)c->max_batch * n_q * c->n_q_heads * c->head_dim * 4, 256);
    s += align_up((size_t)c->max_batch * 64 * 16, 256);
    off += s;
  }
  v.total = off;
  return v;
}

int device_sm_count(int device, int* sms) {
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return SPACE_E_NO_DEVICE;
  if (prop.major != 10) return SPACE_E_NO_DEVICE;
  *sms = prop.multiProcessorCount;
  return SPACE_OK;
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

void build_layout(int k, int variant, space_layout_t* out) {
  memset(out, 0, sizeof(*out));
  const int k1 = k + 1, n = k1 * k1;
  out->k = k; out->n_q = n;
  for (int i = 0; i < n; ++i) {
    const int gi = i / k1, oi = i % k1;
    out->kind[i] = oi != 0; out->group[i] = (uint8_t)gi; out->offset[i] = (uint8_t)oi;
    uint64_t m = 0;
    for (int j = 0; j <= i; ++j) {
      const int gj = j / k1, oj = j % k1;
      bool vis;
      if (oj == 0) vis = true;                         // Eq. 5 case 1: earlier real token
      else if (oi == 0) vis = false;                   // real tokens never see mask tokens
      else if (variant == SPACE_MASK_EQ5_LITERAL) vis = (i - j) < k;    // Eq. 5 case 2 as printed
      else vis = (gi == gj);                           // masks of the same group, causal
      if (vis) m |= 1ull << j;
    }
    out->mask[i] = m;
    out->relpos[i] = __builtin_popcountll(m) - 1;      // Sec. 3.2: visible keys - 1, relative to L
  }
  for (int t = 0; t <= k; ++t) out->target_rows[t] = t * k1;
}

// Every entry point that takes a context makes the context's device current.
bool use_device(const space_ctx* ctx) { return cudaSetDevice(ctx->cfg.device) == cudaSuccess; }

int check_verify_args(const space_ctx* ctx, const space_verify_args* a) {
  if (a->batch < 0 || a->batch > ctx->cfg.max_batch) return SPACE_E_WORKSPACE;
  if (a->k < 1 || a->k > ctx->cfg.k_max) return SPACE_E_INVALID_ARG;
  if (a->vocab < 1 || a->vocab > ctx->cfg.vocab) return SPACE_E_WORKSPACE;
  if (a->batch == 0) return SPACE_OK;
  if (!a->logits || !a->cand || !a->cand_prob || !a->n_accept || !a->out_tokens || !a->n_out ||
      !a->next_cand || !a->next_cand_prob || !a->finished)
    return SPACE_E_INVALID_ARG;
  if (a->logits_dtype != SPACE_DTYPE_F32 && a->logits_dtype != SPACE_DTYPE_BF16) return SPACE_E_INVALID_ARG;
  if (a->mode != SPACE_MODE_GREEDY && a->mode != SPACE_MODE_SAMPLE) return SPACE_E_INVALID_ARG;
  if (a->resample != SPACE_RESAMPLE_RESIDUAL_POINTMASS && a->resample != SPACE_RESAMPLE_PAPER_LITERAL &&
      a->resample != SPACE_RESAMPLE_RESIDUAL_DRAFT)
    return SPACE_E_INVALID_ARG;
  if (a->mode == SPACE_MODE_SAMPLE && a->resample == SPACE_RESAMPLE_RESIDUAL_DRAFT) {
    // compact draft lists are the filtered mask rows: they need a top-k, a place to go, and come in pairs
    if (a->top_k < 1 || !a->next_draft_tok || !a->next_draft_prob) return SPACE_E_INVALID_ARG;
    if ((a->draft_tok == nullptr) != (a->draft_prob == nullptr)) return SPACE_E_INVALID_ARG;
  }
  if (a->mode == SPACE_MODE_SAMPLE && !(a->temperature > 0.f)) return SPACE_E_INVALID_ARG;
  if (a->mode == SPACE_MODE_SAMPLE && a->top_k != 0 &&
      (a->top_k < 0 || a->top_k > 32 || !(a->top_p > 0.f) || a->top_p > 1.f))
    return SPACE_E_INVALID_ARG;
  if (a->logits_row_stride < a->vocab) return SPACE_E_INVALID_ARG;
  const int esz = a->logits_dtype == SPACE_DTYPE_F32 ? 4 : 2;
  if ((uintptr_t)a->logits % esz) return SPACE_E_ALIGNMENT;
  return SPACE_OK;
}

int check_commit_args(const space_ctx* ctx, const space_commit_args* a) {
  if (a->batch < 0 || a->batch > ctx->cfg.max_batch) return SPACE_E_WORKSPACE;
  if (a->k < 1 || a->k > ctx->cfg.k_max) return SPACE_E_INVALID_ARG;
  if (a->batch == 0) return SPACE_OK;
  if (!a->k_cache || !a->v_cache || !a->n_accept || !a->kv_len) return SPACE_E_INVALID_ARG;
  if (!aligned16(a->k_cache) || !aligned16(a->v_cache)) return SPACE_E_ALIGNMENT;
  if (a->kv_stride_b % 8 || a->kv_stride_h % 8 || a->kv_stride_s % 8) return SPACE_E_ALIGNMENT;
  if (a->kv_stride_s < ctx->cfg.head_dim) return SPACE_E_INVALID_ARG;
  if (a->page_table && (a->pages_per_seq < 1 || a->n_pages < 1 ||
                        (int64_t)a->pages_per_seq * SPACE_PAGE_SIZE > ctx->cfg.s_cap))
    return SPACE_E_INVALID_ARG;
  return SPACE_OK;
}

// Test hook kernel: one mbarrier that nothing ever arrives on, waited for with the bounded wait
// every tensor-core kernel of the library uses.  The wait gives up after limit_ns, the kernel
// reports what it saw and returns normally: nothing faults, traps or spins without a bound.
__global__ void wait_timeout_kernel(unsigned long long limit_ns, int32_t* out) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x != 0) return;
  abort_flag = 0;
  const uint32_t b = tc::smem_u32(&bar);
  tc::mbar_init(b, 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  int* err = out + 1;                                       // first time-out site (zeroed by the host)
  const unsigned long long t0 = tc::global_ns();
  const bool ok = tc::mbar_wait_bounded(b, 0, &abort_flag, err, 77, limit_ns, 64);
  const unsigned long long t1 = tc::global_ns();
  const bool again = tc::mbar_wait_bounded(b, 0, &abort_flag, err, 78, limit_ns, 64);   // draining: returns at once
  const unsigned long long t2 = tc::global_ns();
  out[0] = (ok ? 0 : SPACE_ST_TIMEOUT) | (again ? 8 : 0) | (abort_flag ? 16 : 0);
  out[2] = (int32_t)((t1 - t0) / 1000ull);                  // microseconds the first wait took
  out[3] = (int32_t)((t2 - t1) / 1000ull);                  // and the second
}

}  // namespace

extern "C" {

size_t space_workspace_bytes(const space_config* cfg) {
  if (!config_ok(cfg) || config_supported(cfg) != SPACE_OK) return 0;
  return carve(cfg, 148).total;
}

int space_create(space_ctx** out, const space_config* cfg) {
  if (!out) return SPACE_E_INVALID_ARG;
  *out = nullptr;
  if (!config_ok(cfg)) return SPACE_E_INVALID_ARG;
  int rc = config_supported(cfg);
  if (rc != SPACE_OK) return rc;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || cfg->device < 0 || cfg->device >= n_dev) {
    cudaGetLastError();
    return SPACE_E_NO_DEVICE;
  }
  int sms = 0;
  rc = device_sm_count(cfg->device, &sms);
  if (rc != SPACE_OK) return rc;
  if (cudaSetDevice(cfg->device) != cudaSuccess) return SPACE_E_CUDA;
  space_ctx* ctx = new (std::nothrow) space_ctx();
  if (!ctx) return SPACE_E_WORKSPACE;
  memset(ctx, 0, sizeof(*ctx));
  ctx->cfg = *cfg;
  ctx->sm_count = sms;
  const Carve cv = carve(cfg, sms);
  if (cudaMalloc((void**)&ctx->ws, cv.total) != cudaSuccess) {
    cudaGetLastError();
    delete ctx;
    return SPACE_E_WORKSPACE;
  }
  ctx->ws_bytes = cv.total;
  ctx->attn_part = (float*)(ctx->ws + cv.attn_part);
  ctx->attn_part_slots = cv.part_slots;
  ctx->counters = (int*)(ctx->ws + cv.counters);
  ctx->merge_cnt = (int*)(ctx->ws + cv.merge_cnt);
  ctx->vpart = (VerifyPartial*)(ctx->ws + cv.vpart);
  ctx->vtopk = ctx->ws + cv.vtopk;
  ctx->vrow = (VerifyRow*)(ctx->ws + cv.vrow);
  ctx->vfused = (VerifyPartial*)(ctx->ws + cv.vfused);
  ctx->scratch_status = (int32_t*)(ctx->ws + cv.status);
  ctx->lm_part = ctx->ws + cv.lm_part;
  ctx->lm_counter = (int*)(ctx->ws + cv.lm_counter);
  ctx->stage = cfg->host_staging ? ctx->ws + cv.stage : nullptr;
  ctx->stage_bytes = cv.total - cv.stage;
  ctx->host_small = nullptr;
  if (cfg->host_staging &&
      cudaHostAlloc((void**)&ctx->host_small, (size_t)cfg->max_batch * 64 * 11, cudaHostAllocDefault) != cudaSuccess) {
    cudaGetLastError();
    cudaFree(ctx->ws);
    delete ctx;
    return SPACE_E_CUDA;
  }
  if (cfg->host_staging) {
    bool ok = cudaStreamCreateWithFlags(&ctx->aux_stream, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; i < 4 && ok; ++i) ok = cudaEventCreateWithFlags(&ctx->aux_ev[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
      cudaGetLastError();
      if (ctx->host_small) cudaFreeHost(ctx->host_small);
      cudaFree(ctx->ws);
      delete ctx;
      return SPACE_E_CUDA;
    }
  }
  // counters and status start at zero; the kernels restore them after use
  if (cudaMemset(ctx->ws + cv.counters, 0, cv.stage - cv.counters) != cudaSuccess) {
    if (ctx->host_small) cudaFreeHost(ctx->host_small);
    cudaFree(ctx->ws);
    delete ctx;
    return SPACE_E_CUDA;
  }
  *out = ctx;
  return SPACE_OK;
}

void space_destroy(space_ctx* ctx) {
  if (!ctx) return;
  cudaSetDevice(ctx->cfg.device);
  for (int w = 0; w < SPACE_K_COUNT; ++w) {
    if (!ctx->prof_ev[w]) continue;
    for (int i = 0; i < 2 * SPACE_PROFILE_MAX_STEPS; ++i) cudaEventDestroy(ctx->prof_ev[w][i]);
    free(ctx->prof_ev[w]);
  }
  if (ctx->host_small) cudaFreeHost(ctx->host_small);
  if (ctx->aux_stream) {
    for (int i = 0; i < 4; ++i) if (ctx->aux_ev[i]) cudaEventDestroy(ctx->aux_ev[i]);
    cudaStreamDestroy(ctx->aux_stream);
  }
  cudaFree(ctx->ws);
  delete ctx;
}

int space_layout(int k, int mask_variant, space_layout_t* out) {
  if (!out || k < 1 || k > SPACE_MAX_K) return SPACE_E_INVALID_ARG;
  if (mask_variant != SPACE_MASK_SAME_GROUP && mask_variant != SPACE_MASK_EQ5_LITERAL)
    return SPACE_E_INVALID_ARG;
  build_layout(k, mask_variant, out);
  return SPACE_OK;
}

int space_attn_step(space_ctx* ctx, const space_attn_args* a, void* stream) {
  if (!ctx || !a) return SPACE_E_INVALID_ARG;
  if (a->batch < 0 || a->batch > ctx->cfg.max_batch) return SPACE_E_WORKSPACE;
  if (a->k < 1 || a->k > ctx->cfg.k_max) return SPACE_E_INVALID_ARG;
  if (a->batch == 0) return SPACE_OK;
  if (!a->q || !a->k_cache || !a->v_cache || !a->kv_len || !a->out) return SPACE_E_INVALID_ARG;
  if (!(a->scale > 0.f)) return SPACE_E_INVALID_ARG;
  if (a->out_dtype != SPACE_DTYPE_F32 && a->out_dtype != SPACE_DTYPE_BF16) return SPACE_E_INVALID_ARG;
  if (a->mask_variant != SPACE_MASK_SAME_GROUP && a->mask_variant != SPACE_MASK_EQ5_LITERAL)
    return SPACE_E_INVALID_ARG;
  if (!aligned16(a->q) || !aligned16(a->k_cache) || !aligned16(a->v_cache) || !aligned16(a->out))
    return SPACE_E_ALIGNMENT;
  if (a->kv_stride_s < ctx->cfg.head_dim || a->kv_stride_b < 1 || a->kv_stride_h < 1) return SPACE_E_INVALID_ARG;
  if (a->kv_stride_b % 8 || a->kv_stride_h % 8 || a->kv_stride_s % 8) return SPACE_E_ALIGNMENT;
  if (a->page_table && (a->pages_per_seq < 1 || a->n_pages < 1 ||
                        (int64_t)a->pages_per_seq * SPACE_PAGE_SIZE > ctx->cfg.s_cap))
    return SPACE_E_INVALID_ARG;
  if (!use_device(ctx)) return SPACE_E_CUDA;
  if (ctx->lay_k != a->k || ctx->lay_variant != a->mask_variant) {   // the layout is rebuilt only when k or the reading changes
    space_layout_t lay;
    build_layout(a->k, a->mask_variant, &lay);
    memcpy(ctx->lay_mask, lay.mask, sizeof(ctx->lay_mask));
    ctx->lay_k = a->k; ctx->lay_variant = a->mask_variant;
  }
  cudaStream_t st = (cudaStream_t)stream;
  if (a->impl == SPACE_ATTN_SIMT) return launch_attn_simt(ctx, a, ctx->lay_mask, st);
  if (a->impl != SPACE_ATTN_TENSOR && a->impl != SPACE_ATTN_TENSOR_ROWS) return SPACE_E_INVALID_ARG;
  return launch_attn_tensor(ctx, a, ctx->lay_mask, st);
}

int space_verify(space_ctx* ctx, const space_verify_args* a, void* stream) {
  if (!ctx || !a) return SPACE_E_INVALID_ARG;
  const int rc = check_verify_args(ctx, a);
  if (rc != SPACE_OK || a->batch == 0) return rc;
  if (!use_device(ctx)) return SPACE_E_CUDA;
  return launch_verify(ctx, a, nullptr, (cudaStream_t)stream);
}

int space_verify_commit(space_ctx* ctx, const space_verify_args* a, const space_commit_args* c, void* stream) {
  if (!ctx || !a || !c) return SPACE_E_INVALID_ARG;
  int rc = check_verify_args(ctx, a);
  if (rc != SPACE_OK) return rc;
  rc = check_commit_args(ctx, c);
  if (rc != SPACE_OK) return rc;
  if (c->batch != a->batch || c->k != a->k || c->n_accept != a->n_accept) return SPACE_E_INVALID_ARG;
  if (a->batch == 0) return SPACE_OK;
  if (!use_device(ctx)) return SPACE_E_CUDA;
  return launch_verify(ctx, a, c, (cudaStream_t)stream);
}

int space_verify_greedy_noalloc(const space_verify_args* a, void* stream) {
  if (!a) return SPACE_E_INVALID_ARG;
  if (a->batch < 0 || a->k < 1 || a->k > SPACE_MAX_K || a->vocab < 1) return SPACE_E_INVALID_ARG;
  if (a->batch > SPACE_NOALLOC_MAX_BATCH) return SPACE_E_STATIC_LIMIT;
  if (a->batch == 0) return SPACE_OK;
  if (a->mode != SPACE_MODE_GREEDY) return SPACE_E_INVALID_ARG;
  if (!a->logits || !a->cand || !a->cand_prob || !a->n_accept || !a->out_tokens || !a->n_out ||
      !a->next_cand || !a->next_cand_prob || !a->finished)
    return SPACE_E_INVALID_ARG;
  if (a->logits_dtype != SPACE_DTYPE_F32 && a->logits_dtype != SPACE_DTYPE_BF16) return SPACE_E_INVALID_ARG;
  if (a->logits_row_stride < a->vocab) return SPACE_E_INVALID_ARG;
  const int esz = a->logits_dtype == SPACE_DTYPE_F32 ? 4 : 2;
  if ((uintptr_t)a->logits % esz) return SPACE_E_ALIGNMENT;
  return launch_verify_noalloc(a, (cudaStream_t)stream);
}

int space_lmhead_verify(space_ctx* ctx, const space_lmhead_args* a, void* stream) {
  if (!ctx || !a) return SPACE_E_INVALID_ARG;
  if (a->batch < 1 || a->batch > ctx->cfg.max_batch || a->k < 1 || a->k > ctx->cfg.k_max) return SPACE_E_WORKSPACE;
  if (a->vocab < 1 || a->hidden_dim < 8) return SPACE_E_INVALID_ARG;
  if (!a->hidden || !a->weight || !a->cand || !a->n_accept || !a->out_tokens || !a->n_out || !a->next_cand ||
      !a->next_cand_prob || !a->finished)
    return SPACE_E_INVALID_ARG;
  if (a->hidden_dim % 8 || a->hidden_row_stride % 8 || a->weight_row_stride % 8 ||
      ((uintptr_t)a->hidden & 15) || ((uintptr_t)a->weight & 15))
    return SPACE_E_ALIGNMENT;
  if (a->hidden_row_stride < a->hidden_dim || a->weight_row_stride < a->hidden_dim) return SPACE_E_INVALID_ARG;
  if (a->mode != SPACE_MODE_GREEDY && a->mode != SPACE_MODE_SAMPLE) return SPACE_E_INVALID_ARG;
  if (a->mode == SPACE_MODE_SAMPLE) {
    if (!(a->temperature > 0.f) || !a->cand_prob) return SPACE_E_INVALID_ARG;
    if (a->resample != SPACE_RESAMPLE_RESIDUAL_POINTMASS && a->resample != SPACE_RESAMPLE_PAPER_LITERAL)
      return SPACE_E_INVALID_ARG;
  }
  if (!use_device(ctx)) return SPACE_E_CUDA;
  return launch_lmhead_verify(ctx, a, (cudaStream_t)stream);
}

int space_kv_commit(space_ctx* ctx, const space_commit_args* a, void* stream) {
  if (!ctx || !a) return SPACE_E_INVALID_ARG;
  const int rc = check_commit_args(ctx, a);
  if (rc != SPACE_OK || a->batch == 0) return rc;
  if (!use_device(ctx)) return SPACE_E_CUDA;
  return launch_commit(ctx, a, (cudaStream_t)stream);
}

int space_step_host(space_ctx* ctx, const space_host_step_args* a, void* stream) {
  if (!ctx || !a) return SPACE_E_INVALID_ARG;
  if (!ctx->stage) return SPACE_E_WORKSPACE;
  const space_config& c = ctx->cfg;
  if (a->batch < 1 || a->batch > c.max_batch || a->k < 1 || a->k > c.k_max || a->vocab < 1 ||
      a->vocab > c.vocab)
    return SPACE_E_WORKSPACE;
  if (!a->q || !a->k_cache || !a->v_cache || !a->logits || !a->cand || !a->cand_prob || !a->kv_len ||
      !a->out || !a->n_accept || !a->out_tokens || !a->n_out || !a->next_cand || !a->next_cand_prob ||
      !a->finished || !a->status)
    return SPACE_E_INVALID_ARG;
  if (!use_device(ctx)) return SPACE_E_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  const int B = a->batch, k = a->k, k1 = k + 1, n_q = k1 * k1, d = c.head_dim;
  const Carve cv = carve(&c, ctx->sm_count);
  char* sg = ctx->stage;
  char* d_q = sg + cv.st_q; char* d_k = sg + cv.st_k; char* d_v = sg + cv.st_v;
  char* d_logits = sg + cv.st_logits;
  char* d_out = sg + cv.st_small;
  char* d_small = d_out + align_up((size_t)c.max_batch * (size_t)(c.k_max + 1) * (c.k_max + 1) * c.n_q_heads * d * 4, 256);
  // small arrays, 64 bytes-per-sequence slots
  const size_t slot = (size_t)c.max_batch * 64;
  int32_t* d_kvlen = (int32_t*)(d_small);
  int32_t* d_cand = (int32_t*)(d_small + slot);
  float* d_cprob = (float*)(d_small + 2 * slot);
  int32_t* d_nacc = (int32_t*)(d_small + 3 * slot);
  int32_t* d_tok = (int32_t*)(d_small + 4 * slot);
  int32_t* d_nout = (int32_t*)(d_small + 5 * slot);
  int32_t* d_ncand = (int32_t*)(d_small + 6 * slot);
  float* d_nprob = (float*)(d_small + 7 * slot);
  uint8_t* d_fin = (uint8_t*)(d_small + 8 * slot);
  int32_t* d_status = (int32_t*)(d_small + 9 * slot);
  int32_t* d_kvlen_out = (int32_t*)(d_small + 10 * slot);

  int64_t h2d = 0, d2h = 0;
  auto up = [&](void* dst, const void* src, size_t n) {
    h2d += (int64_t)n;
    return cudaMemcpyAsync(dst, src, n, cudaMemcpyHostToDevice, st) == cudaSuccess;
  };
  bool ok = true;
  const size_t row_b = (size_t)d * 2, head_pitch = (size_t)c.s_cap * row_b;
  const size_t seq_b = (size_t)c.n_kv_heads * head_pitch;
  const int esz = a->logits_dtype == SPACE_DTYPE_F32 ? 4 : 2;
  // Two streams: what attention needs (q, the K/V rows, the lengths) goes up first on `st`; the logits
  // follow on the second stream while attention already runs; the attention output comes down on the
  // second stream while verification runs.  Events order the two; the call ends with everything done.
  cudaStream_t sb = ctx->aux_stream;
  ok = ok && up(d_q, a->q, (size_t)B * n_q * c.n_q_heads * d * 2);
  // the small per-sequence arrays travel as one block each way through a pinned mirror of their slots
  char* hsm = ctx->host_small;
  memcpy(hsm, a->kv_len, (size_t)B * 4);
  memcpy(hsm + slot, a->cand, (size_t)B * k * 4);
  memcpy(hsm + 2 * slot, a->cand_prob, (size_t)B * k * 4);
  ok = ok && cudaMemcpyAsync(d_small, hsm, 3 * slot, cudaMemcpyHostToDevice, st) == cudaSuccess;
  h2d += (int64_t)B * 4 * (1 + 2 * k);
  for (int b = 0; b < B && ok; ++b) {
    const int64_t L = a->kv_len[b];
    if (L < 0 || L + n_q > c.s_cap) continue;            // flagged by the kernels
    // everything in use, or (cache kept from an earlier call) the block's own rows only
    const size_t first = a->cache_resident ? (size_t)L * row_b : 0;
    const size_t w = (size_t)(L + n_q) * row_b - first;
    ok = ok && cudaMemcpy2DAsync(d_k + b * seq_b + first, head_pitch, (const char*)a->k_cache + b * seq_b + first,
                                 head_pitch, w, c.n_kv_heads, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok = ok && cudaMemcpy2DAsync(d_v + b * seq_b + first, head_pitch, (const char*)a->v_cache + b * seq_b + first,
                                 head_pitch, w, c.n_kv_heads, cudaMemcpyHostToDevice, st) == cudaSuccess;
    h2d += 2 * (int64_t)w * c.n_kv_heads;
  }
  ok = ok && cudaMemsetAsync(d_status, 0, (size_t)B * 4, st) == cudaSuccess;
  ok = ok && cudaEventRecord(ctx->aux_ev[0], st) == cudaSuccess;          // attention's inputs are on their way
  ok = ok && cudaStreamWaitEvent(sb, ctx->aux_ev[0], 0) == cudaSuccess;
  h2d += (int64_t)((size_t)B * n_q * a->vocab * esz);
  ok = ok && cudaMemcpyAsync(d_logits, a->logits, (size_t)B * n_q * a->vocab * esz, cudaMemcpyHostToDevice, sb) == cudaSuccess;
  ok = ok && cudaEventRecord(ctx->aux_ev[1], sb) == cudaSuccess;          // logits uploaded
  if (!ok) { cudaGetLastError(); return SPACE_E_CUDA; }

  space_attn_args at{};
  at.batch = B; at.k = k; at.mask_variant = a->mask_variant; at.out_dtype = SPACE_DTYPE_F32;
  at.impl = SPACE_ATTN_TENSOR; at.scale = a->scale;
  at.q = d_q; at.k_cache = d_k; at.v_cache = d_v;
  at.kv_stride_b = (int64_t)c.n_kv_heads * c.s_cap * d; at.kv_stride_h = c.s_cap * d; at.kv_stride_s = d;
  at.kv_len = d_kvlen; at.out = d_out; at.lse = nullptr; at.status = d_status;
  int rc = space_attn_step(ctx, &at, stream);
  if (rc != SPACE_OK) return rc;
  // the attention output leaves on the second stream, under the verification kernels
  ok = ok && cudaEventRecord(ctx->aux_ev[2], st) == cudaSuccess;
  ok = ok && cudaStreamWaitEvent(sb, ctx->aux_ev[2], 0) == cudaSuccess;
  d2h += (int64_t)((size_t)B * n_q * c.n_q_heads * d * 4);
  ok = ok && cudaMemcpyAsync(a->out, d_out, (size_t)B * n_q * c.n_q_heads * d * 4, cudaMemcpyDeviceToHost, sb) == cudaSuccess;
  ok = ok && cudaEventRecord(ctx->aux_ev[3], sb) == cudaSuccess;
  ok = ok && cudaStreamWaitEvent(st, ctx->aux_ev[1], 0) == cudaSuccess;   // verification needs the logits
  if (!ok) { cudaGetLastError(); return SPACE_E_CUDA; }
  space_verify_args ve{};
  ve.batch = B; ve.k = k; ve.vocab = a->vocab; ve.logits_dtype = a->logits_dtype; ve.mode = a->mode;
  ve.resample = a->resample; ve.eos_id = a->eos_id; ve.temperature = a->temperature; ve.seed = a->seed;
  ve.logits = d_logits; ve.logits_row_stride = a->vocab; ve.cand = d_cand; ve.cand_prob = d_cprob;
  ve.seq_id = nullptr; ve.kv_len = d_kvlen; ve.n_accept = d_nacc; ve.out_tokens = d_tok; ve.n_out = d_nout;
  ve.next_cand = d_ncand; ve.next_cand_prob = d_nprob; ve.finished = d_fin; ve.status = d_status;
  space_commit_args cm{};
  cm.batch = B; cm.k = k; cm.k_cache = d_k; cm.v_cache = d_v;
  cm.kv_stride_b = at.kv_stride_b; cm.kv_stride_h = at.kv_stride_h; cm.kv_stride_s = at.kv_stride_s;
  cm.n_accept = d_nacc; cm.kv_len = d_kvlen; cm.kv_len_out = d_kvlen_out; cm.status = d_status;
  rc = space_verify_commit(ctx, &ve, &cm, stream);
  if (rc != SPACE_OK) return rc;

  ok = ok && cudaMemcpyAsync(hsm + 3 * slot, d_small + 3 * slot, 8 * slot, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  d2h += (int64_t)B * (4 + k1 * 4 + 4 + k * 4 + k * 4 + 1 + 4 + 4);
  for (int b = 0; b < B && ok; ++b) {                    // rows L .. L+k: the compacted rows
    const int64_t L = a->kv_len[b];
    if (L < 0 || L + n_q > c.s_cap) continue;
    const size_t offb = b * seq_b + (size_t)L * row_b, w = (size_t)k1 * row_b;
    ok = ok && cudaMemcpy2DAsync((char*)a->k_cache + offb, head_pitch, d_k + offb, head_pitch, w, c.n_kv_heads,
                                 cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok = ok && cudaMemcpy2DAsync((char*)a->v_cache + offb, head_pitch, d_v + offb, head_pitch, w, c.n_kv_heads,
                                 cudaMemcpyDeviceToHost, st) == cudaSuccess;
    d2h += 2 * (int64_t)w * c.n_kv_heads;
  }
  ok = ok && cudaStreamWaitEvent(st, ctx->aux_ev[3], 0) == cudaSuccess;   // ... and the output has arrived
  if (!ok) { cudaGetLastError(); return SPACE_E_CUDA; }
  if (cudaStreamSynchronize(st) != cudaSuccess) return SPACE_E_CUDA;
  memcpy(a->n_accept, hsm + 3 * slot, (size_t)B * 4);
  memcpy(a->out_tokens, hsm + 4 * slot, (size_t)B * k1 * 4);
  memcpy(a->n_out, hsm + 5 * slot, (size_t)B * 4);
  memcpy(a->next_cand, hsm + 6 * slot, (size_t)B * k * 4);
  memcpy(a->next_cand_prob, hsm + 7 * slot, (size_t)B * k * 4);
  memcpy(a->finished, hsm + 8 * slot, (size_t)B);
  memcpy(a->status, hsm + 9 * slot, (size_t)B * 4);
  memcpy(a->kv_len, hsm + 10 * slot, (size_t)B * 4);
  if (a->h2d_bytes) *a->h2d_bytes = h2d;
  if (a->d2h_bytes) *a->d2h_bytes = d2h;
  return SPACE_OK;
}

int64_t space_launch_count(const space_ctx* ctx) { return ctx ? ctx->launches : 0; }

int space_profile_enable(space_ctx* ctx, int on) {
  if (!ctx) return SPACE_E_INVALID_ARG;
  if (on) {
    for (int w = 0; w < SPACE_K_COUNT; ++w) {
      if (!ctx->prof_ev[w]) {
        cudaEvent_t* ev = (cudaEvent_t*)calloc(2 * SPACE_PROFILE_MAX_STEPS, sizeof(cudaEvent_t));
        if (!ev) return SPACE_E_WORKSPACE;
        for (int i = 0; i < 2 * SPACE_PROFILE_MAX_STEPS; ++i)
          if (cudaEventCreate(&ev[i]) != cudaSuccess) { free(ev); return SPACE_E_CUDA; }
        ctx->prof_ev[w] = ev;
      }
      ctx->prof_n[w] = 0;
    }
  }
  ctx->prof_on = on != 0;
  return SPACE_OK;
}

int space_profile_read(space_ctx* ctx, float* ms, int64_t* n) {
  if (!ctx || !ms || !n) return SPACE_E_INVALID_ARG;
  for (int w = 0; w < SPACE_K_COUNT; ++w) {
    double sum = 0.0;
    for (int i = 0; i < ctx->prof_n[w]; ++i) {
      float t = 0.f;
      if (cudaEventSynchronize(ctx->prof_ev[w][2 * i + 1]) != cudaSuccess ||
          cudaEventElapsedTime(&t, ctx->prof_ev[w][2 * i], ctx->prof_ev[w][2 * i + 1]) != cudaSuccess)
        return SPACE_E_CUDA;
      sum += t;
    }
    ms[w] = (float)sum;
    n[w] = ctx->prof_n[w];
    ctx->prof_n[w] = 0;
  }
  return SPACE_OK;
}

int space_debug_philox(space_ctx* ctx, uint64_t seed, int64_t n, const uint32_t* c0, const uint32_t* c1,
                       const uint32_t* c2, const uint32_t* c3, uint32_t* out, void* stream) {
  if (!ctx || n < 0 || (n > 0 && (!c0 || !c1 || !c2 || !c3 || !out))) return SPACE_E_INVALID_ARG;
  if (!use_device(ctx)) return SPACE_E_CUDA;
  return launch_philox_debug(seed, n, c0, c1, c2, c3, out, (cudaStream_t)stream);
}

int space_debug_wait_timeout(space_ctx* ctx, uint64_t limit_ns, int32_t* out4, void* stream) {
  if (!ctx || !out4 || limit_ns == 0 || limit_ns > 100000000ull) return SPACE_E_INVALID_ARG;   // at most 0.1 s
  if (!use_device(ctx)) return SPACE_E_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemsetAsync(out4, 0, 4 * sizeof(int32_t), st) != cudaSuccess) return SPACE_E_CUDA;
  wait_timeout_kernel<<<1, 32, 0, st>>>((unsigned long long)limit_ns, out4);
  return cuda_ok(cudaGetLastError());
}

const char* space_strerror(int code) {
  switch (code) {
    case SPACE_OK: return "ok";
    case SPACE_E_INVALID_ARG: return "invalid argument";
    case SPACE_E_UNSUPPORTED: return "shape not supported by the kernels";
    case SPACE_E_ALIGNMENT: return "pointer or stride not 16-byte aligned";
    case SPACE_E_WORKSPACE: return "request exceeds the workspace reserved by space_create";
    case SPACE_E_CUDA: return "CUDA call failed";
    case SPACE_E_NO_DEVICE: return "no usable sm_100 device";
    case SPACE_E_STATIC_LIMIT: return "batch exceeds the fixed scratch of space_verify_greedy_noalloc (SPACE_NOALLOC_MAX_BATCH)";
    default: return "unknown error";
  }
}

}  // extern "C"
