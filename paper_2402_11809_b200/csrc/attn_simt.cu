// Plain SIMT attention of the block rows over cache + block (Eq. 5): one
// thread block per (sequence, query head, block row), fp32 CUDA-core
// arithmetic, no tensor cores, no splitting.  It exists as an in-library
// cross-check of the tensor-core kernel (space_attn_args.impl =
// SPACE_ATTN_SIMT); it is far from the memory roofline.
#include "common.cuh"
#include <math_constants.h>

namespace {

struct SimtParams {
  int B, k, n_q, H_q, H_kv, d, out_dtype;
  int64_t s_cap;
  float scale;
  const __nv_bfloat16* q; const __nv_bfloat16* kc; const __nv_bfloat16* vc;
  int64_t sb, sh, ss;
  const int32_t* kv_len;
  void* out; float* lse; int32_t* status;
  uint64_t mask[SPACE_MAX_ROWS];
  const int32_t* page_table; int pages_per_seq, n_pages;   // paged cache, or page_table == nullptr
};

constexpr int SIMT_THREADS = 128;

__device__ float block_max(float v, float* sh) {
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = sh[0];
  for (int i = 1; i < SIMT_THREADS / 32; ++i) r = fmaxf(r, sh[i]);
  __syncthreads();
  return r;
}

__device__ float block_sum(float v, float* sh) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = 0.f;
  for (int i = 0; i < SIMT_THREADS / 32; ++i) r += sh[i];
  __syncthreads();
  return r;
}

__global__ void __launch_bounds__(SIMT_THREADS) attn_simt_kernel(const SimtParams p) {
  extern __shared__ float smem[];          // [d] query, then scores
  __shared__ float red[SIMT_THREADS / 32];
  const int i = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int L = p.kv_len[b];
  if (L < 0 || (int64_t)L + p.n_q > p.s_cap) {
    if (threadIdx.x == 0 && i == 0 && h == 0 && p.status) atomicOr(p.status + b, SPACE_ST_CAPACITY);
    return;
  }
  const int hk = h / (p.H_q / p.H_kv);
  float* qs = smem;
  float* sc = smem + p.d;
  const __nv_bfloat16* qrow = p.q + (((int64_t)b * p.n_q + i) * p.H_q + h) * p.d;
  for (int c = threadIdx.x; c < p.d; c += SIMT_THREADS) qs[c] = __bfloat162float(qrow[c]);
  __syncthreads();
  // offset of key row j (contiguous cache, or through the page table); a page outside the pool
  // reads as zeros and is flagged
  __shared__ int bad_page;
  if (threadIdx.x == 0) bad_page = 0;
  __syncthreads();
  auto row_off = [&](int j) {
    const int64_t o = kv_row_offset(p.page_table, p.pages_per_seq, p.n_pages, p.sb, p.sh, p.ss, b, hk, j);
    if (o < 0) bad_page = 1;
    return o;
  };
  const int n_keys = L + p.n_q;
  const uint64_t mrow = p.mask[i];
  float mx = -CUDART_INF_F;
  for (int j = threadIdx.x; j < n_keys; j += SIMT_THREADS) {
    const bool vis = (j < L) || ((mrow >> (j - L)) & 1ull);
    float s = -CUDART_INF_F;
    if (vis) {
      const int64_t ko = row_off(j);
      const __nv_bfloat162* kr = reinterpret_cast<const __nv_bfloat162*>(p.kc + (ko < 0 ? 0 : ko));
      float acc = 0.f;
      for (int c = 0; c < (ko < 0 ? 0 : p.d / 2); ++c) {
        const float2 kk = __bfloat1622float2(kr[c]);
        acc = fmaf(qs[2 * c], kk.x, acc);
        acc = fmaf(qs[2 * c + 1], kk.y, acc);
      }
      s = acc * p.scale;
    }
    sc[j] = s;
    mx = fmaxf(mx, s);
  }
  mx = block_max(mx, red);
  float sum = 0.f;
  for (int j = threadIdx.x; j < n_keys; j += SIMT_THREADS) {
    const float e = (sc[j] > -CUDART_INF_F) ? __expf(sc[j] - mx) : 0.f;
    sc[j] = e;
    sum += e;
  }
  sum = block_sum(sum, red);
  const float inv = 1.f / sum;
  for (int c = threadIdx.x; c < p.d; c += SIMT_THREADS) {
    float acc = 0.f;
    for (int j = 0; j < n_keys; ++j) {
      const float e = sc[j];
      if (e != 0.f) {
        const int64_t vo = row_off(j);
        if (vo >= 0) acc = fmaf(e, __bfloat162float(p.vc[vo + c]), acc);
      }
    }
    const int64_t o = (((int64_t)b * p.n_q + i) * p.H_q + h) * p.d + c;
    if (p.out_dtype == SPACE_DTYPE_F32) reinterpret_cast<float*>(p.out)[o] = acc * inv;
    else reinterpret_cast<__nv_bfloat16*>(p.out)[o] = __float2bfloat16_rn(acc * inv);
  }
  if (p.lse && threadIdx.x == 0) p.lse[((int64_t)b * p.H_q + h) * p.n_q + i] = mx + logf(sum);
  __syncthreads();
  if (threadIdx.x == 0 && bad_page && p.status) atomicOr(p.status + b, SPACE_ST_BAD_PAGE);
}

}  // namespace

int launch_attn_simt(space_ctx* ctx, const space_attn_args* a, const uint64_t* mask_rows,
                     cudaStream_t st) {
  SimtParams p;
  p.B = a->batch; p.k = a->k; p.n_q = (a->k + 1) * (a->k + 1);
  p.H_q = ctx->cfg.n_q_heads; p.H_kv = ctx->cfg.n_kv_heads; p.d = ctx->cfg.head_dim;
  p.out_dtype = a->out_dtype; p.scale = a->scale;
  p.s_cap = a->page_table ? (int64_t)a->pages_per_seq * SPACE_PAGE_SIZE : ctx->cfg.s_cap;
  p.page_table = a->page_table; p.pages_per_seq = a->pages_per_seq; p.n_pages = a->n_pages;
  p.q = (const __nv_bfloat16*)a->q; p.kc = (const __nv_bfloat16*)a->k_cache;
  p.vc = (const __nv_bfloat16*)a->v_cache;
  p.sb = a->kv_stride_b; p.sh = a->kv_stride_h; p.ss = a->kv_stride_s;
  p.kv_len = a->kv_len; p.out = a->out; p.lse = a->lse; p.status = a->status;
  for (int i = 0; i < SPACE_MAX_ROWS; ++i) p.mask[i] = mask_rows[i];
  const size_t smem = (size_t)(p.d + ctx->cfg.s_cap) * sizeof(float);
  if (smem > 200 * 1024) return SPACE_E_UNSUPPORTED;
  cudaFuncSetAttribute(attn_simt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  {
    ProfScope ps(ctx, SPACE_K_ATTN, st);
    attn_simt_kernel<<<dim3(p.n_q, p.H_q, p.B), SIMT_THREADS, smem, st>>>(p);
  }
  ctx->launches += 1;
  return cuda_ok(cudaGetLastError());
}
