// dlm_guided_accept: the Guided Diffusion accept rule (Sec. 3.2.2, Algorithm 1).
//
// Integer-only and tiny (one block of positions per batch element), so it is bound by launch
// latency.  One warp per batch element walks the block 32 positions at a time; ballots give
// the masked set, the first disagreement and the ascending output order without any sort.
#include "common.cuh"

namespace {

__global__ void __launch_bounds__(32)
guided_accept_kernel(const int32_t* __restrict__ tok_dlm, const int32_t* __restrict__ tok_ar, int top_k, int block_len,
                     uint8_t* __restrict__ masked, int32_t* __restrict__ tokens, int fallback_source,
                     uint8_t* __restrict__ accept, int32_t* __restrict__ acc_idx, int32_t* __restrict__ n_acc) {
  dlm_grid_dependency_wait();
  dlm_trigger_dependents();
  const int b = blockIdx.x;
  const int lane = threadIdx.x;
  const size_t o = (size_t)b * block_len;
  const unsigned lt_mask = (1u << lane) - 1u;
  int n = 0;             // accepted so far (warp-uniform)
  int first_masked = -1; // i_1
  bool open = true;      // still inside the agreeing prefix
  for (int base = 0; base < block_len; base += 32) {
    const int i = base + lane;
    const bool in = i < block_len;
    const bool m = in && masked[o + i] != 0;
    const int td = in ? tok_dlm[o + i] : 0;
    // agreement: the DLM token is among the guider's top_k tokens for this position (top_k = 1: its argmax)
    bool agree = false;
    if (m) {
      const int32_t* cand = tok_ar + (o + i) * top_k;
      for (int j = 0; j < top_k; ++j) agree = agree || cand[j] == td;
    }
    const unsigned mm = __ballot_sync(0xffffffffu, m);
    const unsigned dis = __ballot_sync(0xffffffffu, m && !agree);
    if (first_masked < 0 && mm) first_masked = base + __ffs(mm) - 1;
    bool mine = false;
    if (open) {
      const unsigned below_first_dis = dis ? ((1u << (__ffs(dis) - 1)) - 1u) : 0xffffffffu;
      const unsigned acc = mm & below_first_dis;
      mine = (acc >> lane) & 1u;
      if (mine) {
        acc_idx[o + n + __popc(acc & lt_mask)] = i;
        tokens[o + i] = td;
        masked[o + i] = 0;
      }
      n += __popc(acc);
      if (dis) open = false;
    }
    if (in) accept[o + i] = mine ? 1 : 0;
  }
  __syncwarp();
  if (n == 0 && first_masked >= 0) {  // no agreement at i_1: accept it alone
    if (lane == 0) {
      const size_t q = o + first_masked;
      accept[q] = 1;
      acc_idx[o] = first_masked;
      tokens[q] = fallback_source == 1 ? tok_ar[q * top_k] : tok_dlm[q];
      masked[q] = 0;
    }
    n = 1;
  }
  for (int j = n + lane; j < block_len; j += 32) acc_idx[o + j] = -1;
  if (lane == 0) n_acc[b] = n;
}

// The accept rule with the confidence threshold (App. C.3 "Stochastic Guided Unmasking"): the Top-K match result
// above (fallback included) united with every masked position whose largest DLM logit exceeds tau times the largest
// of the guider's top_k logits for it.  Same walk as above; the accepted set need not be a prefix any more.
__global__ void __launch_bounds__(32)
guided_accept_threshold_kernel(const int32_t* __restrict__ tok_dlm, const float* __restrict__ zmax_dlm,
                               const int32_t* __restrict__ tok_ar, const float* __restrict__ logit_ar, int top_k, float tau,
                               int block_len, uint8_t* __restrict__ masked, int32_t* __restrict__ tokens,
                               int fallback_source, uint8_t* __restrict__ accept, int32_t* __restrict__ acc_idx,
                               int32_t* __restrict__ n_acc) {
  dlm_grid_dependency_wait();
  dlm_trigger_dependents();
  const int b = blockIdx.x;
  const int lane = threadIdx.x;
  const size_t o = (size_t)b * block_len;
  const unsigned lt_mask = (1u << lane) - 1u;
  int n = 0;             // accepted so far (warp-uniform)
  bool seen_masked = false;
  bool open = true;      // still inside the agreeing prefix
  for (int base = 0; base < block_len; base += 32) {
    const int i = base + lane;
    const bool in = i < block_len;
    const bool m = in && masked[o + i] != 0;
    const int td = in ? tok_dlm[o + i] : 0;
    bool agree = false, pass = false;
    if (m) {
      const int32_t* cand = tok_ar + (o + i) * top_k;
      const float* lg = logit_ar + (o + i) * top_k;
      float g = lg[0];
      for (int j = 0; j < top_k; ++j) {
        agree = agree || cand[j] == td;
        g = fmaxf(g, lg[j]);
      }
      pass = zmax_dlm[o + i] > tau * g;
    }
    const unsigned mm = __ballot_sync(0xffffffffu, m);
    const unsigned dis = __ballot_sync(0xffffffffu, m && !agree);
    unsigned acc = __ballot_sync(0xffffffffu, m && pass);
    bool lone_fallback = false;   // this lane holds i_1, accepted by the fallback alone
    if (open) {
      const unsigned below_first_dis = dis ? ((1u << (__ffs(dis) - 1)) - 1u) : 0xffffffffu;
      acc |= mm & below_first_dis;
      if (!seen_masked && mm) {
        const int first = __ffs(mm) - 1;
        if ((dis >> first) & 1u) {   // no agreement at i_1: it is accepted whatever else happens
          lone_fallback = lane == first && !pass;
          acc |= 1u << first;
        }
      }
      if (dis) open = false;
    }
    if (mm) seen_masked = true;
    const bool mine = (acc >> lane) & 1u;
    if (mine) {
      acc_idx[o + n + __popc(acc & lt_mask)] = i;
      tokens[o + i] = (lone_fallback && fallback_source == 1) ? tok_ar[(o + i) * top_k] : td;
      masked[o + i] = 0;
    }
    n += __popc(acc);
    if (in) accept[o + i] = mine ? 1 : 0;
  }
  for (int j = n + lane; j < block_len; j += 32) acc_idx[o + j] = -1;
  if (lane == 0) n_acc[b] = n;
}

}  // namespace

extern "C" int dlm_guided_accept(dlm_ctx* ctx, const int32_t* tok_dlm, const int32_t* tok_ar, int batch,
                                 int block_len, uint8_t* masked, int32_t* tokens, int fallback_source,
                                 uint8_t* accept, int32_t* acc_idx, int32_t* n_acc, void* stream) {
  if (!ctx || !tok_dlm || !tok_ar || !masked || !tokens || !accept || !acc_idx || !n_acc) return DLM_ERR_NULL;
  if (batch <= 0 || block_len <= 0) return DLM_ERR_SHAPE;
  if (block_len > 1024 || (fallback_source != 0 && fallback_source != 1)) return DLM_ERR_UNSUPPORTED;
  DLM_DEVICE_TRY(ctx);
  DLM_CUDA_TRY(dlm_launch(guided_accept_kernel, dim3(batch), dim3(32), 0, static_cast<cudaStream_t>(stream), tok_dlm, tok_ar, 1,
                          block_len, masked, tokens, fallback_source, accept, acc_idx, n_acc));
  return dlm_launch_ok(ctx, 1);
}

extern "C" int dlm_guided_accept_topk(dlm_ctx* ctx, const int32_t* tok_dlm, const int32_t* tok_ar_topk, int top_k,
                                      int batch, int block_len, uint8_t* masked, int32_t* tokens, int fallback_source,
                                      uint8_t* accept, int32_t* acc_idx, int32_t* n_acc, void* stream) {
  if (!ctx || !tok_dlm || !tok_ar_topk || !masked || !tokens || !accept || !acc_idx || !n_acc) return DLM_ERR_NULL;
  if (batch <= 0 || block_len <= 0 || top_k <= 0) return DLM_ERR_SHAPE;
  if (block_len > 1024 || top_k > 64 || (fallback_source != 0 && fallback_source != 1)) return DLM_ERR_UNSUPPORTED;
  DLM_DEVICE_TRY(ctx);
  DLM_CUDA_TRY(dlm_launch(guided_accept_kernel, dim3(batch), dim3(32), 0, static_cast<cudaStream_t>(stream), tok_dlm,
                          tok_ar_topk, top_k, block_len, masked, tokens, fallback_source, accept, acc_idx, n_acc));
  return dlm_launch_ok(ctx, 1);
}

extern "C" int dlm_guided_accept_threshold(dlm_ctx* ctx, const int32_t* tok_dlm, const float* zmax_dlm,
                                           const int32_t* tok_ar_topk, const float* logit_ar_topk, int top_k, float tau,
                                           int batch, int block_len, uint8_t* masked, int32_t* tokens,
                                           int fallback_source, uint8_t* accept, int32_t* acc_idx, int32_t* n_acc,
                                           void* stream) {
  if (!ctx || !tok_dlm || !zmax_dlm || !tok_ar_topk || !logit_ar_topk || !masked || !tokens || !accept || !acc_idx || !n_acc)
    return DLM_ERR_NULL;
  if (batch <= 0 || block_len <= 0 || top_k <= 0) return DLM_ERR_SHAPE;
  if (block_len > 1024 || top_k > 64 || (fallback_source != 0 && fallback_source != 1) || !(tau == tau))
    return DLM_ERR_UNSUPPORTED;
  DLM_DEVICE_TRY(ctx);
  DLM_CUDA_TRY(dlm_launch(guided_accept_threshold_kernel, dim3(batch), dim3(32), 0, static_cast<cudaStream_t>(stream), tok_dlm,
                          zmax_dlm, tok_ar_topk, logit_ar_topk, top_k, tau, block_len, masked, tokens, fallback_source, accept,
                          acc_idx, n_acc));
  return dlm_launch_ok(ctx, 1);
}
