// Sample transform of semi-autoregressive fine-tuning (Sec. 3.1, App. A.1) on a padded batch.
//
// With probability 1 - p_ar a sample's k answer tokens from a random position m on are replaced
// by the mask token in the input (the labels stay) and input and labels are cut after the first
// m + k answer tokens; otherwise the sample is left as it is.  The random decisions are taken
// from two 32-bit words per sample in integer arithmetic: the sample stays autoregressive when
// the first word is below ar_threshold, and m = (second word * (N - k + 1)) >> 32.
// One thread block per sample.
#include "common.cuh"

namespace {

__global__ void __launch_bounds__(128) sar_sft_kernel(const space_sar_args a) {
  const int b = blockIdx.x;
  const int P = a.prompt_len[b], N = a.answer_len[b];
  const uint32_t w0 = a.rand_words[2 * b], w1 = a.rand_words[2 * b + 1];
  const bool ar = w0 < a.ar_threshold || N < a.k || P < 0 || N < 0 || (int64_t)P + N > a.seq_cap;
  if (ar) {
    if (threadIdx.x == 0) {
      if (a.new_len) a.new_len[b] = P + N;
      if (a.mask_start) a.mask_start[b] = -1;
    }
    return;
  }
  const int m = (int)(((uint64_t)w1 * (uint64_t)(N - a.k + 1)) >> 32);   // uniform on {0, .., N-k}
  const int keep = P + m + a.k;
  int32_t* ids = a.input_ids + (int64_t)b * a.seq_cap;
  int32_t* lab = a.labels + (int64_t)b * a.seq_cap;
  for (int i = P + m + threadIdx.x; i < a.seq_cap; i += blockDim.x) {
    if (i < keep) ids[i] = a.mask_token_id;                // the k masked answer tokens
    else { ids[i] = a.pad_token_id; lab[i] = a.ignore_index; }   // cut: beyond m + k answer tokens
  }
  if (threadIdx.x == 0) {
    if (a.new_len) a.new_len[b] = keep;
    if (a.mask_start) a.mask_start[b] = m;
  }
}

}  // namespace

extern "C" int space_sar_sft_transform(const space_sar_args* a, void* stream) {
  if (!a) return SPACE_E_INVALID_ARG;
  if (a->batch < 0 || a->seq_cap < 1 || a->k < 1) return SPACE_E_INVALID_ARG;
  if (a->batch == 0) return SPACE_OK;
  if (!a->input_ids || !a->labels || !a->prompt_len || !a->answer_len || !a->rand_words) return SPACE_E_INVALID_ARG;
  sar_sft_kernel<<<a->batch, 128, 0, (cudaStream_t)stream>>>(*a);
  return cuda_ok(cudaGetLastError());
}
