// Greedy acceptance of a draft tree (Sec. 4.2: the original model verifies the drafted tokens and accepts or rejects
// them).  One warp per sequence; lane l decides nodes l and l + 32 by walking their ancestors -- a node is accepted
// when every token on its path equals the verifier's arg-max token at the node before it -- and the warp then picks
// the deepest accepted node, the smallest index among equally deep ones.  Integer work only.
#include "la_common.cuh"

namespace la {

constexpr int kAcceptWarps = 4;   // sequences per CTA

__global__ void __launch_bounds__(32 * kAcceptWarps)
accept_greedy_kernel(const int32_t* __restrict__ parent, const int32_t* __restrict__ draft, const int32_t* __restrict__ pred_root,
                     const int32_t* __restrict__ pred, int32_t* __restrict__ accept_node, int32_t* __restrict__ accept_len,
                     int32_t* __restrict__ next_token, int* status, int B, int N) {
  __shared__ int s_par[kAcceptWarps][LA_MAX_NODES], s_draft[kAcceptWarps][LA_MAX_NODES], s_pred[kAcceptWarps][LA_MAX_NODES];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x * kAcceptWarps + warp;
  if (b >= B) return;                                  // whole warps leave: no block-wide barrier below
  for (int n = lane; n < N; n += 32) {
    s_par[warp][n] = parent[(size_t)b * N + n];
    s_draft[warp][n] = draft[(size_t)b * N + n];
    s_pred[warp][n] = pred[(size_t)b * N + n];
  }
  const int root = pred_root[b];
  __syncwarp();

  bool bad = false;
  int best_key = 0;                                    // depth * 64 + (63 - node): larger is better; 0 = none
  for (int n = lane; n < N; n += 32) {
    int m = n, depth = 0;
    bool acc = true;
    while (m >= 0) {                                   // m strictly decreases: at most N iterations
      const int p = s_par[warp][m];
      if (p < -1 || p >= m) { bad = true; break; }
      acc = acc && s_draft[warp][m] == (p < 0 ? root : s_pred[warp][p]);
      ++depth;
      m = p;
    }
    if (acc && !bad) best_key = max(best_key, depth * 64 + (63 - n));
  }
  bad = __any_sync(0xffffffffu, bad);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) best_key = max(best_key, __shfl_xor_sync(0xffffffffu, best_key, o));
  if (lane == 0) {
    if (bad) {
      report(status, LA_ERR_BAD_TREE);
      best_key = 0;
    }
    const int node = best_key ? 63 - (best_key & 63) : -1;
    accept_node[b] = node;
    accept_len[b] = best_key >> 6;
    if (next_token) next_token[b] = node >= 0 ? s_pred[warp][node] : root;
  }
}

// Acceptance by a per-node score and threshold (Sec. 4.2: the original model accepts or rejects the drafted tokens,
// resampling if needed).  A node passes when score >= threshold (a comparison with a NaN fails) and is accepted when
// every node on its path passes; the caller brings the scores and thresholds of whichever rule it samples by (the
// ratio p/q against a uniform draw; the probability against an entropy bound).  Same walk, same choice as above.
__global__ void __launch_bounds__(32 * kAcceptWarps)
accept_threshold_kernel(const int32_t* __restrict__ parent, const float* __restrict__ score, const float* __restrict__ thresh,
                        int32_t* __restrict__ accept_node, int32_t* __restrict__ accept_len, int* status, int B, int N) {
  __shared__ int s_par[kAcceptWarps][LA_MAX_NODES];
  __shared__ unsigned char s_pass[kAcceptWarps][LA_MAX_NODES];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x * kAcceptWarps + warp;
  if (b >= B) return;                                  // whole warps leave: no block-wide barrier below
  for (int n = lane; n < N; n += 32) {
    s_par[warp][n] = parent[(size_t)b * N + n];
    s_pass[warp][n] = score[(size_t)b * N + n] >= thresh[(size_t)b * N + n] ? 1 : 0;
  }
  __syncwarp();

  bool bad = false;
  int best_key = 0;                                    // depth * 64 + (63 - node): larger is better; 0 = none
  for (int n = lane; n < N; n += 32) {
    int m = n, depth = 0;
    bool acc = true;
    while (m >= 0) {                                   // m strictly decreases: at most N iterations
      const int p = s_par[warp][m];
      if (p < -1 || p >= m) { bad = true; break; }
      acc = acc && s_pass[warp][m] != 0;
      ++depth;
      m = p;
    }
    if (acc && !bad) best_key = max(best_key, depth * 64 + (63 - n));
  }
  bad = __any_sync(0xffffffffu, bad);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) best_key = max(best_key, __shfl_xor_sync(0xffffffffu, best_key, o));
  if (lane == 0) {
    if (bad) {
      report(status, LA_ERR_BAD_TREE);
      best_key = 0;
    }
    accept_node[b] = best_key ? 63 - (best_key & 63) : -1;
    accept_len[b] = best_key >> 6;
  }
}

cudaError_t launch_accept_threshold(la_ctx* ctx, int B, int N, const int32_t* parent, const float* score, const float* thresh,
                                    int32_t* accept_node, int32_t* accept_len, cudaStream_t s) {
  accept_threshold_kernel<<<dim3((B + kAcceptWarps - 1) / kAcceptWarps), dim3(32 * kAcceptWarps), 0, s>>>(
      parent, score, thresh, accept_node, accept_len, ctx->d_status, B, N);
  ctx->launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_accept(la_ctx* ctx, int B, int N, const int32_t* parent, const int32_t* draft, const int32_t* pred_root,
                          const int32_t* pred, int32_t* accept_node, int32_t* accept_len, int32_t* next_token,
                          cudaStream_t s) {
  accept_greedy_kernel<<<dim3((B + kAcceptWarps - 1) / kAcceptWarps), dim3(32 * kAcceptWarps), 0, s>>>(
      parent, draft, pred_root, pred, accept_node, accept_len, next_token, ctx->d_status, B, N);
  ctx->launches += 1;
  return cudaGetLastError();
}

}  // namespace la
