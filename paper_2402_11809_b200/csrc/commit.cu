// KV-commit kernel: compaction of the accepted rows into the verified cache.
//
// Algorithm 1 re-runs the model on the whole sequence each step and therefore
// has no cache; with one, the rows that join the verified prefix are the root
// and the accepted candidates: block rows g(k+1), g = 0..i*, which move from
// cache position L + g(k+1) to L + g.  Destinations L+1..L+k are mask rows of
// sub-block 0 and never a source, so the move is safe in place.
#include "common.cuh"

namespace {

__global__ void __launch_bounds__(256) kv_commit_kernel(const CommitParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.y, part = blockIdx.x;
  const int L = p.kv_len[b];
  int i_star = p.n_accept[b];
  i_star = max(0, min(i_star, p.k));
  const bool fits = commit_fits(p, L);
  if (fits) commit_rows_any(p, b, L, i_star, part, p.blocks_per_seq, threadIdx.x, blockDim.x);
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
  commit_tables(p, b, L, i_star, fits);
}

}  // namespace

void fill_commit_params(const space_ctx* ctx, const space_commit_args* a, CommitParams* pp) {
  CommitParams& p = *pp;
  p.B = a->batch; p.k = a->k; p.H_kv = ctx->cfg.n_kv_heads; p.d = ctx->cfg.head_dim;
  p.s_cap = a->page_table ? (int64_t)a->pages_per_seq * SPACE_PAGE_SIZE : ctx->cfg.s_cap;
  p.page_table = a->page_table; p.pages_per_seq = a->pages_per_seq; p.n_pages = a->n_pages;
  p.kc = (__nv_bfloat16*)a->k_cache; p.vc = (__nv_bfloat16*)a->v_cache;
  p.sb = a->kv_stride_b; p.sh = a->kv_stride_h; p.ss = a->kv_stride_s;
  p.n_accept = a->n_accept; p.kv_len = a->kv_len; p.kv_len_out = a->kv_len_out;
  p.src = a->commit_src; p.dst = a->commit_dst; p.status = a->status;
  p.counter = ctx->counters + 2 * ctx->cfg.max_batch;
  p.in_place = (a->kv_len_out == a->kv_len);
  p.blocks_per_seq = 1;
}

int launch_commit(space_ctx* ctx, const space_commit_args* a, cudaStream_t st) {
  CommitParams p;
  fill_commit_params(ctx, a, &p);
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
