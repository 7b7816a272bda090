// Shared declarations of the CUDA sources: context, launchers, small device
// helpers.  Internal to the library; the public contract is include/falcon.h.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "falcon.h"

struct falcon_ctx {
  int device = 0;
  int sm_count = 0;
  int smem_optin = 0;
  // Scratch shared by all calls on this context (split partials, argmax partials).
  void* ws = nullptr;
  size_t ws_bytes = 0;
  // Arrival counters; zero between calls (the last arriver resets its counter).
  int* tickets = nullptr;
  size_t n_tickets = 0;
  // Scratch blocks that were outgrown.  A launch already enqueued, or captured into a CUDA graph,
  // may still name them, so they live until falcon_destroy.
  std::vector<void*> retired;
  std::string last_error;
  // Cached TMA descriptors (opaque here; owned by tc_util.cuh).
  void* tmap_cache = nullptr;
  // Per-context launch state of the tensor-core attention kernels: whether the dynamic shared
  // memory limit has been raised on this device, and how many clusters of each size fit at once
  // (0 = not asked yet, -1 = none).  Index 0: rows-on-lanes kernel; 1-3: the keys-on-lanes kernel's
  // three variants.
  bool attn_attr_set[4] = {false, false, false, false};
  bool lm_attr_set = false;  // the same for the LM-head kernel
  int attn_resident[4][9] = {};
};

namespace falcon {

int ensure_workspace(falcon_ctx* ctx, size_t bytes);
int ensure_tickets(falcon_ctx* ctx, size_t count, cudaStream_t stream);
int cuda_fail(falcon_ctx* ctx, cudaError_t e, const char* where);
int check_tree_desc(const falcon_tree_desc& t, bool need_token);

// launchers (one per kernel file)
int launch_tree_accept(falcon_ctx* ctx, const falcon_accept_args& a, cudaStream_t s);
int launch_kv_compact(falcon_ctx* ctx, const falcon_compact_args& a, cudaStream_t s);
int launch_feature_gather(falcon_ctx* ctx, const falcon_gather_args& a, cudaStream_t s);
int check_gather_args(const falcon_gather_args& g, int max_tree);
int launch_tree_topm(falcon_ctx* ctx, const falcon_topm_args& a, cudaStream_t s);
int launch_test_poison(falcon_ctx* ctx, uint32_t pattern, cudaStream_t s);
int launch_tree_search(falcon_ctx* ctx, const falcon_accept_args& a, cudaStream_t s);
int launch_tree_sample(falcon_ctx* ctx, const falcon_accept_args& a, cudaStream_t s);
int launch_lm_head_argmax(falcon_ctx* ctx, const falcon_lm_argmax_args& a, cudaStream_t s);
int launch_tree_attn_simt(falcon_ctx* ctx, const falcon_attn_args& a, cudaStream_t s);
int launch_tree_attn_tc(falcon_ctx* ctx, const falcon_attn_args& a, cudaStream_t s);
bool tree_attn_tc_supports(const falcon_ctx* ctx, const falcon_attn_args& a);
int launch_tree_attn_tck(falcon_ctx* ctx, const falcon_attn_args& a, cudaStream_t s);
bool tree_attn_tck_supports(const falcon_ctx* ctx, const falcon_attn_args& a);
bool tree_attn_tck_preferred(const falcon_ctx* ctx, const falcon_attn_args& a);
int launch_tree_attn_warp(falcon_ctx* ctx, const falcon_attn_args& a, cudaStream_t s);
bool tree_attn_warp_supports(const falcon_ctx* ctx, const falcon_attn_args& a);
void tree_attn_tc_release(falcon_ctx* ctx);

#ifdef __CUDACC__
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ void dev_status_or(int32_t* status, int b, int bits) {
  if (status != nullptr) atomicOr(&status[b], bits);
}

// Bit t of a 128-bit set stored as two 64-bit words.
__device__ __forceinline__ bool bit128(uint64_t lo, uint64_t hi, int t) {
  return ((t < 64 ? lo >> t : hi >> (t - 64)) & 1ull) != 0;
}

// Ancestor-or-self set of node i as a 128-bit mask, by walking the parent
// array.  The walk is capped at T steps; a parent outside [0, u) ends it.
// Returns false when the tree is malformed.
__device__ __forceinline__ bool ancestor_mask(const int32_t* __restrict__ parent, int T, int i, uint64_t& lo,
                                              uint64_t& hi) {
  lo = 0;
  hi = 0;
  int u = i;
  bool ok = true;
  for (int step = 0; step < T; ++step) {
    if (u < 64) lo |= 1ull << u; else hi |= 1ull << (u - 64);
    if (u == 0) break;
    const int pu = parent[u];
    if (pu < 0 || pu >= u) { ok = false; break; }
    u = pu;
  }
  return ok;
}
#endif

}  // namespace falcon
