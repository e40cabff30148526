// C boundary: argument validation, dispatch to the kernel launchers, status handling.
#include <cmath>
#include <cstdlib>
#include <new>

#include "la_common.cuh"

namespace {

// A launcher's error as a status: a shape the tensor-core path covers on a driver that cannot encode tensor maps is
// LA_ERR_UNSUPPORTED (there is no silent detour over the CUDA-core kernels), everything else LA_ERR_CUDA.
inline la_status cuda_status(cudaError_t e) {
  return e == cudaSuccess ? LA_OK : e == cudaErrorNotSupported ? LA_ERR_UNSUPPORTED : LA_ERR_CUDA;
}
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool good(const void* p) { return p != nullptr && aligned16(p); }

bool state_ok(const la_ctx* ctx, const la_state* st) {
  if (!st || !good(st->S) || !good(st->z) || st->pos == nullptr) return false;
  if (ctx->cfg.conv_taps > 1 && !good(st->win)) return false;
  return true;
}

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    if (prev == dev) prev = -1;
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

}  // namespace

extern "C" {

const char* la_status_str(la_status s) {
  switch (s) {
    case LA_OK: return "LA_OK";
    case LA_ERR_INVALID_ARG: return "LA_ERR_INVALID_ARG";
    case LA_ERR_UNSUPPORTED: return "LA_ERR_UNSUPPORTED";
    case LA_ERR_CUDA: return "LA_ERR_CUDA";
    case LA_ERR_BAD_TREE: return "LA_ERR_BAD_TREE";
    case LA_ERR_TIMEOUT: return "LA_ERR_TIMEOUT";
    case LA_ERR_TOO_LARGE: return "LA_ERR_TOO_LARGE";
  }
  return "LA_ERR_UNKNOWN";
}

la_status la_create(const la_config* cfg, la_ctx** out) {
  if (!cfg || !out) return LA_ERR_INVALID_ARG;
  *out = nullptr;
  if (cfg->H < 1 || cfg->conv_taps < 1 || cfg->conv_taps > LA_MAX_TAPS || cfg->chunk < 0) return LA_ERR_INVALID_ARG;
  if (cfg->phi != LA_PHI_ELU1 && cfg->phi != LA_PHI_RELU) return LA_ERR_INVALID_ARG;
  if (cfg->io_dtype != LA_F32 && cfg->io_dtype != LA_BF16) return LA_ERR_INVALID_ARG;
  if (!(cfg->eps >= 0.f) || !std::isfinite(cfg->eps)) return LA_ERR_INVALID_ARG;
  if (cfg->max_nodes < 1 || cfg->max_nodes > LA_MAX_NODES) return LA_ERR_INVALID_ARG;
  if (cfg->max_depth < 1 || cfg->max_depth > LA_MAX_NODES) return LA_ERR_INVALID_ARG;
  if (cfg->d != 64 && cfg->d != 128) return LA_ERR_UNSUPPORTED;

  la_ctx* ctx = new (std::nothrow) la_ctx();
  if (!ctx) return LA_ERR_CUDA;
  ctx->cfg = *cfg;
  ctx->prefill_kernel = 0;
  ctx->launches = 0;
  ctx->d_status = nullptr;
  ctx->ws = nullptr;
  ctx->ws_bytes = 0;
  if (cudaGetDevice(&ctx->device) != cudaSuccess ||
      cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device) != cudaSuccess ||
      cudaMalloc(&ctx->d_status, sizeof(int)) != cudaSuccess ||
      cudaMemset(ctx->d_status, 0, sizeof(int)) != cudaSuccess) {
    if (ctx->d_status) cudaFree(ctx->d_status);
    delete ctx;
    cudaGetLastError();
    return LA_ERR_CUDA;
  }
  *out = ctx;
  return LA_OK;
}

la_status la_destroy(la_ctx* ctx) {
  if (!ctx) return LA_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  cudaError_t e = cudaFree(ctx->d_status);
  delete ctx;
  return e == cudaSuccess ? LA_OK : LA_ERR_CUDA;
}

la_status la_set_prefill_kernel(la_ctx* ctx, int32_t which) {
  if (!ctx || which < 0 || which > 1) return LA_ERR_INVALID_ARG;
  ctx->prefill_kernel = which;
  return LA_OK;
}

int64_t la_launch_count(const la_ctx* ctx) { return ctx ? ctx->launches : -1; }

la_status la_set_workspace(la_ctx* ctx, void* workspace, uint64_t bytes) {
  if (!ctx || (workspace == nullptr) != (bytes == 0) || !aligned16(workspace)) return LA_ERR_INVALID_ARG;
  ctx->ws = workspace;
  ctx->ws_bytes = bytes;
  return LA_OK;
}

uint64_t la_prefill_workspace_bytes(const la_ctx* ctx, int32_t B, int32_t T) {
  if (!ctx || B < 1 || T < 1) return 0;
  return la::prefill_workspace_bytes(ctx, B, T);
}

la_status la_prefill(la_ctx* ctx, int32_t B, int32_t T, const void* q, const void* k, const void* v,
                     const float* conv_w, int32_t init_state, la_state* st, void* o, void* stream) {
  if (!ctx || B < 1 || T < 1 || !good(q) || !good(k) || !good(v) || !good(conv_w) || !good(o)) return LA_ERR_INVALID_ARG;
  if (!state_ok(ctx, st) || (init_state != 0 && init_state != 1)) return LA_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return LA_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (ctx->prefill_kernel == 0) {
    bool handled = false;
    cudaError_t e = la::launch_prefill_tc(ctx, B, T, q, k, v, conv_w, init_state, *st, o, s, &handled);
    if (e != cudaSuccess) return cuda_status(e);
    if (handled) return LA_OK;
  }
  return la::launch_prefill_simt(ctx, B, T, q, k, v, conv_w, init_state, *st, o, s) == cudaSuccess ? LA_OK
                                                                                                   : LA_ERR_CUDA;
}

la_status la_prefill_grouped(la_ctx* ctx, int32_t B, int32_t T, const void* q, const void* k, const void* v,
                             const float* conv_w, int32_t group, float alpha, float softmax_scale, int32_t init_state,
                             la_state* st, void* o, void* stream) {
  if (!ctx || B < 1 || T < 1 || !good(q) || !good(k) || !good(v) || !good(conv_w) || !good(o)) return LA_ERR_INVALID_ARG;
  if (!state_ok(ctx, st) || (init_state != 0 && init_state != 1) || group < 1) return LA_ERR_INVALID_ARG;
  if (!std::isfinite(alpha) || !std::isfinite(softmax_scale)) return LA_ERR_INVALID_ARG;
  if (group > la::prefill_grouped_max_group(ctx->cfg)) return LA_ERR_UNSUPPORTED;
  DeviceGuard g(ctx->device);
  if (!g.ok) return LA_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (ctx->prefill_kernel == 0) {
    bool handled = false;
    const cudaError_t e = la::launch_prefill_grouped_tc(ctx, B, T, q, k, v, conv_w, group, alpha, softmax_scale, init_state,
                                                        *st, o, s, &handled);
    if (e != cudaSuccess) return cuda_status(e);
    if (handled) return LA_OK;
  }
  return cuda_status(la::launch_prefill_grouped(ctx, B, T, q, k, v, conv_w, group, alpha, softmax_scale, init_state, *st, o, s));
}

int32_t la_prefill_grouped_max_group(const la_ctx* ctx) { return ctx ? la::prefill_grouped_max_group(ctx->cfg) : 0; }

la_status la_segment_state(la_ctx* ctx, int32_t B, int32_t T, const void* k, const void* v, float* dS, float* dz,
                           void* stream) {
  if (!ctx || B < 1 || T < 1 || !good(k) || !good(v) || !good(dS) || !good(dz)) return LA_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return LA_ERR_CUDA;
  return cuda_status(la::launch_segment_state(ctx, B, T, k, v, dS, dz, static_cast<cudaStream_t>(stream)));
}

la_status la_state_prefix(la_ctx* ctx, int32_t B, int32_t nparts, int32_t count, const float* dS_parts,
                          const float* dz_parts, const float* S_base, const float* z_base, float* S_out, float* z_out,
                          void* stream) {
  if (!ctx || B < 1 || nparts < 1 || count < 0 || count > nparts || !good(dS_parts) || !good(dz_parts) || !good(S_out) ||
      !good(z_out) || (S_base == nullptr) != (z_base == nullptr) || !aligned16(S_base) || !aligned16(z_base))
    return LA_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return LA_ERR_CUDA;
  const size_t nz = (size_t)B * ctx->cfg.H * ctx->cfg.d, nS = nz * ctx->cfg.d;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (la::launch_state_prefix(ctx, dS_parts, S_base, S_out, nS, count, s) != cudaSuccess) return LA_ERR_CUDA;
  return cuda_status(la::launch_state_prefix(ctx, dz_parts, z_base, z_out, nz, count, s));
}

la_status la_decode_step(la_ctx* ctx, int32_t B, const void* q, const void* k, const void* v, const float* conv_w,
                         la_state* st, void* o, void* stream) {
  if (!ctx || B < 1 || !good(q) || !good(k) || !good(v) || !good(conv_w) || !good(o)) return LA_ERR_INVALID_ARG;
  if (!state_ok(ctx, st)) return LA_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return LA_ERR_CUDA;
  return la::launch_decode(ctx, B, q, k, v, conv_w, *st, o, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? LA_OK
             : LA_ERR_CUDA;
}

la_status la_verify_tree(la_ctx* ctx, int32_t B, int32_t N, const void* q, const void* k, const void* v,
                         const int32_t* parent, const float* conv_w, const la_state* st, void* o, void* stream) {
  if (!ctx || B < 1 || N < 1 || !good(q) || !good(k) || !good(v) || !good(conv_w) || !good(o) || !parent)
    return LA_ERR_INVALID_ARG;
  if (N > ctx->cfg.max_nodes) return LA_ERR_INVALID_ARG;
  if (!state_ok(ctx, st)) return LA_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return LA_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (ctx->prefill_kernel == 0) {
    bool handled = false;
    const cudaError_t e = la::launch_verify_tc(ctx, B, N, q, k, v, parent, conv_w, *st, o, s, &handled);
    if (e != cudaSuccess) return cuda_status(e);
    if (handled) return LA_OK;
  }
  return la::launch_verify(ctx, B, N, q, k, v, parent, conv_w, *st, o, s) == cudaSuccess ? LA_OK : LA_ERR_CUDA;
}

la_status la_commit(la_ctx* ctx, int32_t B, int32_t N, const void* k, const void* v, const int32_t* parent,
                    const int32_t* accept_node, la_state* st, int32_t* path_out, int32_t* commit_len, void* stream) {
  if (!ctx || B < 1 || N < 1 || !good(k) || !good(v) || !parent || !accept_node || !path_out || !commit_len)
    return LA_ERR_INVALID_ARG;
  if (N > ctx->cfg.max_nodes) return LA_ERR_INVALID_ARG;
  if (!state_ok(ctx, st)) return LA_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return LA_ERR_CUDA;
  return la::launch_commit(ctx, B, N, k, v, parent, accept_node, *st, path_out, commit_len,
                           static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? LA_OK
             : LA_ERR_CUDA;
}

la_status la_accept_greedy(la_ctx* ctx, int32_t B, int32_t N, const int32_t* parent, const int32_t* draft_token,
                           const int32_t* pred_root, const int32_t* pred, int32_t* accept_node, int32_t* accept_len,
                           int32_t* next_token, void* stream) {
  if (!ctx || B < 1 || N < 1 || !parent || !draft_token || !pred_root || !pred || !accept_node || !accept_len)
    return LA_ERR_INVALID_ARG;
  if (N > ctx->cfg.max_nodes) return LA_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return LA_ERR_CUDA;
  return la::launch_accept(ctx, B, N, parent, draft_token, pred_root, pred, accept_node, accept_len, next_token,
                           static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? LA_OK
             : LA_ERR_CUDA;
}

la_status la_accept_threshold(la_ctx* ctx, int32_t B, int32_t N, const int32_t* parent, const float* score,
                              const float* thresh, int32_t* accept_node, int32_t* accept_len, void* stream) {
  if (!ctx || B < 1 || N < 1 || !parent || !score || !thresh || !accept_node || !accept_len) return LA_ERR_INVALID_ARG;
  if (N > ctx->cfg.max_nodes) return LA_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return LA_ERR_CUDA;
  return la::launch_accept_threshold(ctx, B, N, parent, score, thresh, accept_node, accept_len,
                                     static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? LA_OK
             : LA_ERR_CUDA;
}

la_status la_last_device_status(la_ctx* ctx, void* stream) {
  if (!ctx) return LA_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return LA_ERR_CUDA;
  int code = 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(&code, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess)
    return LA_ERR_CUDA;
  return static_cast<la_status>(code);
}

la_status la_clear_device_status(la_ctx* ctx, void* stream) {
  if (!ctx) return LA_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return LA_ERR_CUDA;
  return cudaMemsetAsync(ctx->d_status, 0, sizeof(int), static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? LA_OK
             : LA_ERR_CUDA;
}

}  // extern "C"
