// C-ABI entry points: argument validation, context management, dispatch.
#include <cstdio>
#include <cstring>
#include <new>

#include "common.cuh"

namespace falcon {

int cuda_fail(falcon_ctx* ctx, cudaError_t e, const char* where) {
  if (ctx) ctx->last_error = std::string(where) + ": " + cudaGetErrorString(e);
  return FALCON_ERR_CUDA;
}

// Scratch only ever grows, and a block that was outgrown is kept until the context is destroyed:
// a kernel already enqueued, or a captured graph, may still name it.
int ensure_workspace(falcon_ctx* ctx, size_t bytes) {
  if (bytes <= ctx->ws_bytes) return FALCON_OK;
  const size_t want = bytes + bytes / 4;
  void* fresh = nullptr;
  cudaError_t e = cudaMalloc(&fresh, want);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaMalloc(workspace)");
  if (ctx->ws) ctx->retired.push_back(ctx->ws);
  ctx->ws = fresh;
  ctx->ws_bytes = want;
  return FALCON_OK;
}

// Arrival counters must read zero when a kernel first uses them: a new block is cleared on the
// caller's stream, ahead of the launch that follows (the kernels leave their counters at zero).
int ensure_tickets(falcon_ctx* ctx, size_t count, cudaStream_t stream) {
  if (count <= ctx->n_tickets) return FALCON_OK;
  const size_t want = count * 2 + 64;
  int* fresh = nullptr;
  cudaError_t e = cudaMalloc(&fresh, want * sizeof(int));
  if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaMalloc(tickets)");
  e = cudaMemsetAsync(fresh, 0, want * sizeof(int), stream);
  if (e != cudaSuccess) {
    cudaFree(fresh);
    return cuda_fail(ctx, e, "cudaMemsetAsync(tickets)");
  }
  if (ctx->tickets) ctx->retired.push_back(ctx->tickets);
  ctx->tickets = fresh;
  ctx->n_tickets = want;
  return FALCON_OK;
}

int check_tree_desc(const falcon_tree_desc& t, bool need_token) {
  if (t.batch < 1 || t.total_nodes < t.batch || t.max_tree < 1 || t.max_prefix_len < 0) return FALCON_ERR_INVALID_ARG;
  if (t.max_tree > FALCON_T_MAX) return FALCON_ERR_UNSUPPORTED;
  if (!t.node_off || !t.parent || !t.prefix_len) return FALCON_ERR_INVALID_ARG;
  if (need_token && !t.token) return FALCON_ERR_INVALID_ARG;
  if (static_cast<int64_t>(t.max_tree) * t.batch < t.total_nodes) return FALCON_ERR_INVALID_ARG;
  return FALCON_OK;
}

}  // namespace falcon

using namespace falcon;

extern "C" {

int falcon_create(falcon_ctx** out, int device) {
  if (!out) return FALCON_ERR_INVALID_ARG;
  *out = nullptr;
  cudaError_t e = cudaSetDevice(device);
  if (e != cudaSuccess) return FALCON_ERR_CUDA;
  cudaDeviceProp prop;
  e = cudaGetDeviceProperties(&prop, device);
  if (e != cudaSuccess) return FALCON_ERR_CUDA;
  if (prop.major != 10) return FALCON_ERR_UNSUPPORTED;  // built for sm_100a only
  falcon_ctx* ctx = new (std::nothrow) falcon_ctx();
  if (!ctx) return FALCON_ERR_INVALID_ARG;
  ctx->device = device;
  ctx->sm_count = prop.multiProcessorCount;
  ctx->smem_optin = static_cast<int>(prop.sharedMemPerBlockOptin);
  *out = ctx;
  return FALCON_OK;
}

int falcon_destroy(falcon_ctx* ctx) {
  if (!ctx) return FALCON_ERR_INVALID_ARG;
  cudaSetDevice(ctx->device);
  tree_attn_tc_release(ctx);
  if (ctx->ws) cudaFree(ctx->ws);
  if (ctx->tickets) cudaFree(ctx->tickets);
  for (void* blk : ctx->retired) cudaFree(blk);
  delete ctx;
  return FALCON_OK;
}

const char* falcon_status_string(int status) {
  switch (status) {
    case FALCON_OK: return "ok";
    case FALCON_ERR_INVALID_ARG: return "invalid argument";
    case FALCON_ERR_UNSUPPORTED: return "unsupported shape or device";
    case FALCON_ERR_CUDA: return "CUDA error";
    case FALCON_ERR_BAD_TREE: return "malformed tree";
    case FALCON_ERR_CAPACITY: return "size exceeds capacity";
    case FALCON_ERR_TIMEOUT: return "device wait timed out";
    default: return "unknown status";
  }
}

const char* falcon_last_error(const falcon_ctx* ctx) { return ctx ? ctx->last_error.c_str() : ""; }

int falcon_tree_validate_host(const int32_t* parent, int32_t T) {
  if (!parent) return FALCON_ERR_INVALID_ARG;
  if (T < 1) return FALCON_ERR_BAD_TREE;
  if (T > FALCON_T_MAX) return FALCON_ERR_UNSUPPORTED;
  if (parent[0] != -1) return FALCON_ERR_BAD_TREE;
  for (int32_t i = 1; i < T; ++i)
    if (parent[i] < 0 || parent[i] >= i) return FALCON_ERR_BAD_TREE;
  return FALCON_OK;
}

// Argument checks of falcon_tree_attn and the kernel it dispatches to; *kernel is one of
// FALCON_ATTN_SIMT / _TC / _TCK on success.
static int attn_plan(falcon_ctx* ctx, const falcon_attn_args* a, int* kernel) {
  if (!ctx || !a) return FALCON_ERR_INVALID_ARG;
  int rc = check_tree_desc(a->tree, false);
  if (rc) return rc;
  if (!a->q || !a->out || !a->k_cache || !a->v_cache) return FALCON_ERR_INVALID_ARG;
  if ((a->k_tree == nullptr) != (a->v_tree == nullptr)) return FALCON_ERR_INVALID_ARG;
  if (a->n_q_heads < 1 || a->n_kv_heads < 1 || a->s_cap < 1) return FALCON_ERR_INVALID_ARG;
  if (a->n_q_heads % a->n_kv_heads != 0) return FALCON_ERR_UNSUPPORTED;
  if (a->head_dim != 64 && a->head_dim != 128) return FALCON_ERR_UNSUPPORTED;
  if (a->kv_stride_s < a->head_dim || a->kv_stride_h < 0 || a->kv_stride_b < 0) return FALCON_ERR_INVALID_ARG;
  if ((a->kv_stride_s | a->kv_stride_h | a->kv_stride_b) & 7) return FALCON_ERR_INVALID_ARG;
  const uintptr_t align = reinterpret_cast<uintptr_t>(a->q) | reinterpret_cast<uintptr_t>(a->out) |
                          reinterpret_cast<uintptr_t>(a->k_cache) | reinterpret_cast<uintptr_t>(a->v_cache) |
                          reinterpret_cast<uintptr_t>(a->k_tree) | reinterpret_cast<uintptr_t>(a->v_tree);
  if (align & 15) return FALCON_ERR_INVALID_ARG;
  if (a->n_splits < 0 || a->n_splits > 64) return FALCON_ERR_INVALID_ARG;
  if (!(a->sm_scale == a->sm_scale)) return FALCON_ERR_INVALID_ARG;
  if ((a->flags & FALCON_ATTN_TEST_STALL) &&
      (a->n_splits != 1 || (a->kernel != FALCON_ATTN_TC && a->kernel != FALCON_ATTN_TCK)))
    return FALCON_ERR_INVALID_ARG;
  switch (a->kernel) {
    case FALCON_ATTN_SIMT:
      *kernel = FALCON_ATTN_SIMT;
      return FALCON_OK;
    case FALCON_ATTN_TC:
      if (!tree_attn_tc_supports(ctx, *a)) return FALCON_ERR_UNSUPPORTED;
      *kernel = FALCON_ATTN_TC;
      return FALCON_OK;
    case FALCON_ATTN_TCK:
      if (!tree_attn_tck_supports(ctx, *a)) return FALCON_ERR_UNSUPPORTED;
      *kernel = FALCON_ATTN_TCK;
      return FALCON_OK;
    case FALCON_ATTN_WARP:
      if (!tree_attn_warp_supports(ctx, *a)) return FALCON_ERR_UNSUPPORTED;
      *kernel = FALCON_ATTN_WARP;
      return FALCON_OK;
    case FALCON_ATTN_AUTO:
      // tensor cores where a kernel takes the shape (which of the two: by shape, measured); else one
      // warp per query row while the scores of a row fit its shared memory; else the tiled kernel
      if (tree_attn_tck_supports(ctx, *a) && (tree_attn_tck_preferred(ctx, *a) || !tree_attn_tc_supports(ctx, *a)))
        *kernel = FALCON_ATTN_TCK;
      else if (tree_attn_tc_supports(ctx, *a))
        *kernel = FALCON_ATTN_TC;
      else if (tree_attn_warp_supports(ctx, *a))
        *kernel = FALCON_ATTN_WARP;
      else
        *kernel = FALCON_ATTN_SIMT;
      return FALCON_OK;
    default:
      return FALCON_ERR_INVALID_ARG;
  }
}

int falcon_test_poison(falcon_ctx* ctx, uint32_t pattern, void* stream) {
  if (!ctx) return FALCON_ERR_INVALID_ARG;
  return launch_test_poison(ctx, pattern, static_cast<cudaStream_t>(stream));
}

int falcon_tree_attn_kernel(falcon_ctx* ctx, const falcon_attn_args* a) {
  int kernel = -1;
  return attn_plan(ctx, a, &kernel) == FALCON_OK ? kernel : -1;
}

int falcon_tree_attn(falcon_ctx* ctx, const falcon_attn_args* a, void* stream) {
  int kernel = -1;
  const int rc = attn_plan(ctx, a, &kernel);
  if (rc) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (kernel == FALCON_ATTN_TCK) return launch_tree_attn_tck(ctx, *a, s);
  if (kernel == FALCON_ATTN_TC) return launch_tree_attn_tc(ctx, *a, s);
  if (kernel == FALCON_ATTN_WARP) return launch_tree_attn_warp(ctx, *a, s);
  return launch_tree_attn_simt(ctx, *a, s);
}

int falcon_tree_accept(falcon_ctx* ctx, const falcon_accept_args* a, void* stream) {
  if (!ctx || !a) return FALCON_ERR_INVALID_ARG;
  int rc = check_tree_desc(a->tree, true);
  if (rc) return rc;
  if (!a->argmax_out || !a->path || !a->n_path || !a->next_token) return FALCON_ERR_INVALID_ARG;
  if (a->path_stride < a->tree.max_tree) return FALCON_ERR_INVALID_ARG;
  if (!(a->temperature >= 0.f)) return FALCON_ERR_INVALID_ARG;
  if (!a->logits) {  // g is given
    if (a->temperature != 0.f) return FALCON_ERR_INVALID_ARG;
    return launch_tree_search(ctx, *a, static_cast<cudaStream_t>(stream));
  }
  if (a->vocab < 1 || a->logits_stride < a->vocab) return FALCON_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(a->logits) & 3) return FALCON_ERR_INVALID_ARG;
  if (a->temperature > 0.f) {
    if (!a->uniforms || (reinterpret_cast<uintptr_t>(a->uniforms) & 3)) return FALCON_ERR_INVALID_ARG;
    return launch_tree_sample(ctx, *a, static_cast<cudaStream_t>(stream));
  }
  return launch_tree_accept(ctx, *a, static_cast<cudaStream_t>(stream));
}

int falcon_lm_head_argmax(falcon_ctx* ctx, const falcon_lm_argmax_args* a, void* stream) {
  if (!ctx || !a) return FALCON_ERR_INVALID_ARG;
  if (!a->features || !a->lm_head || !a->argmax_out) return FALCON_ERR_INVALID_ARG;
  if (a->n_rows < 1 || a->hidden < 1 || a->vocab < 1) return FALCON_ERR_INVALID_ARG;
  if (a->feat_stride < a->hidden || a->head_stride < a->hidden) return FALCON_ERR_INVALID_ARG;
  // TMA: 16-byte aligned bases and row pitches
  if ((a->feat_stride | a->head_stride) & 7) return FALCON_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(a->features) | reinterpret_cast<uintptr_t>(a->lm_head)) & 15) return FALCON_ERR_UNSUPPORTED;
  if (a->n_rows > 65535) return FALCON_ERR_CAPACITY;
  if (a->flags & ~FALCON_LM_TEST_STALL) return FALCON_ERR_INVALID_ARG;
  return launch_lm_head_argmax(ctx, *a, static_cast<cudaStream_t>(stream));
}

int falcon_topm(falcon_ctx* ctx, const falcon_topm_args* a, void* stream) {
  if (!ctx || !a) return FALCON_ERR_INVALID_ARG;
  if (!a->logits || !a->top_val || !a->top_idx) return FALCON_ERR_INVALID_ARG;
  if (a->n_rows < 1 || a->vocab < 1 || a->logits_stride < a->vocab) return FALCON_ERR_INVALID_ARG;
  if (a->m < 1 || a->m > a->vocab || a->m > FALCON_TOPM_MAX) return FALCON_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(a->logits) & 3) return FALCON_ERR_INVALID_ARG;
  if (a->vocab > 64 * 4096) return FALCON_ERR_CAPACITY;
  return launch_tree_topm(ctx, *a, static_cast<cudaStream_t>(stream));
}

int falcon_kv_compact(falcon_ctx* ctx, const falcon_compact_args* a, void* stream) {
  if (!ctx || !a) return FALCON_ERR_INVALID_ARG;
  int rc = check_tree_desc(a->tree, false);
  if (rc) return rc;
  if (!a->k_cache_layers || !a->v_cache_layers || !a->path || !a->n_path || !a->new_len) return FALCON_ERR_INVALID_ARG;
  if ((a->k_tree_layers == nullptr) != (a->v_tree_layers == nullptr)) return FALCON_ERR_INVALID_ARG;
  if (a->n_layers < 1 || a->n_kv_heads < 1 || a->s_cap < 1) return FALCON_ERR_INVALID_ARG;
  if (a->head_dim < 8 || a->head_dim > 256 || (a->head_dim & 7)) return FALCON_ERR_UNSUPPORTED;
  if (a->kv_stride_s < a->head_dim || a->kv_stride_h < 0 || a->kv_stride_b < 0) return FALCON_ERR_INVALID_ARG;
  if ((a->kv_stride_s | a->kv_stride_h | a->kv_stride_b) & 7) return FALCON_ERR_INVALID_ARG;
  if (a->path_stride < a->tree.max_tree) return FALCON_ERR_INVALID_ARG;
  if (a->gather) {
    if (!a->tree.token) return FALCON_ERR_INVALID_ARG;
    rc = check_gather_args(*a->gather, a->tree.max_tree);
    if (rc) return rc;
  }
  return launch_kv_compact(ctx, *a, static_cast<cudaStream_t>(stream));
}

int falcon_feature_gather(falcon_ctx* ctx, const falcon_gather_args* a, void* stream) {
  if (!ctx || !a) return FALCON_ERR_INVALID_ARG;
  int rc = check_tree_desc(a->tree, true);
  if (rc) return rc;
  if (!a->path || !a->n_path || a->path_stride < a->tree.max_tree) return FALCON_ERR_INVALID_ARG;
  rc = check_gather_args(*a, a->tree.max_tree);
  if (rc) return rc;
  return launch_feature_gather(ctx, *a, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
