// KV-commit kernel: compaction of the accepted rows into the verified cache.
//
// Algorithm 1 re-runs the model on the whole sequence each step and therefore
// has no cache; with one, the rows that join the verified prefix are the root
// and the accepted candidates: block rows g(k+1), g = 0..i*, which move from
// cache position L + g(k+1) to L + g.  Destinations L+1..L+k are mask rows of
// sub-block 0 and never a source, so the move is safe in place.
#include "common.cuh"

namespace {

struct CommitParams {
  int B, k, H_kv, d, blocks_per_seq, in_place;
  int64_t s_cap;
  __nv_bfloat16* kc; __nv_bfloat16* vc;
  int64_t sb, sh, ss;
  const int32_t* n_accept; const int32_t* kv_len;
  int32_t* kv_len_out; int32_t* src; int32_t* dst; int32_t* status;
  int* counter;
};

__global__ void __launch_bounds__(256) kv_commit_kernel(const CommitParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.y, part = blockIdx.x;
  const int L = p.kv_len[b];
  int i_star = p.n_accept[b];
  i_star = max(0, min(i_star, p.k));
  const int k1 = p.k + 1;
  const bool fits = (int64_t)L + (int64_t)k1 * k1 <= p.s_cap && L >= 0;
  if (fits) {
    const int vec_per_row = p.d / 8;                    // 16-byte pieces per row
    const int total = i_star * p.H_kv * 2 * vec_per_row;
    for (int t = part * blockDim.x + threadIdx.x; t < total; t += p.blocks_per_seq * blockDim.x) {
      int r = t;
      const int v = r % vec_per_row; r /= vec_per_row;
      const int which = r % 2;       r /= 2;
      const int h = r % p.H_kv;      r /= p.H_kv;
      const int g = r + 1;                              // accepted candidate g = 1..i*
      __nv_bfloat16* base = (which ? p.vc : p.kc) + (int64_t)b * p.sb + (int64_t)h * p.sh;
      const uint4* s = reinterpret_cast<const uint4*>(base + (int64_t)(L + g * k1) * p.ss) + v;
      uint4* dd = reinterpret_cast<uint4*>(base + (int64_t)(L + g) * p.ss) + v;
      *dd = *s;
    }
  }
  // New length and index tables.  When the new length goes to its own array no
  // block depends on another and block 0 writes them at once; when it overwrites
  // kv_len itself the other blocks must have read the old value first, so the
  // last block to arrive (counter, reset for the next launch) writes them.
  if (p.in_place) {
    __shared__ int last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
      const int prev = atomicAdd(p.counter + b, 1);
      last = (prev == p.blocks_per_seq - 1);
      if (last) p.counter[b] = 0;
    }
    __syncthreads();
    if (!last) return;
  } else if (part != 0) {
    return;
  }
  if (threadIdx.x != 0) return;
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

}  // namespace

int launch_commit(space_ctx* ctx, const space_commit_args* a, cudaStream_t st) {
  CommitParams p;
  p.B = a->batch; p.k = a->k; p.H_kv = ctx->cfg.n_kv_heads; p.d = ctx->cfg.head_dim;
  p.s_cap = ctx->cfg.s_cap;
  p.kc = (__nv_bfloat16*)a->k_cache; p.vc = (__nv_bfloat16*)a->v_cache;
  p.sb = a->kv_stride_b; p.sh = a->kv_stride_h; p.ss = a->kv_stride_s;
  p.n_accept = a->n_accept; p.kv_len = a->kv_len; p.kv_len_out = a->kv_len_out;
  p.src = a->commit_src; p.dst = a->commit_dst; p.status = a->status;
  p.counter = ctx->counters + 2 * ctx->cfg.max_batch;
  p.in_place = (a->kv_len_out == a->kv_len);
  // worst case k rows x H_kv heads x K,V x d/8 pieces; one piece per thread, 256 threads
  const int worst = a->k * p.H_kv * 2 * (p.d / 8);
  int blocks = (worst + 255) / 256;
  const int want = (2 * ctx->sm_count + a->batch - 1) / a->batch;
  if (blocks > want) blocks = want;
  if (blocks < 1) blocks = 1;
  p.blocks_per_seq = blocks;
  {
    ProfScope ps(ctx, SPACE_K_COMMIT, st);
    launch_pdl(kv_commit_kernel, dim3(blocks, a->batch), dim3(256), 0, st, p);
  }
  ctx->launches += 1;
  return cuda_ok(cudaGetLastError());
}
