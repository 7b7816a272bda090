// falcon_kv_compact: the accepted path's K/V rows become the contiguous tail of
// the cache, every layer and both K and V in one launch.  One CTA owns all rows
// of one (layer, K|V, sequence, KV head): it reads every source row into
// registers, passes a barrier, then writes, so a destination row that is also an
// earlier source row (in-place mode) cannot be clobbered before it is read.
// Launch/latency-bound byte copy with 16-byte accesses: what matters is that the
// whole grid is resident at once (each CTA is a chain of three dependent round
// trips to memory), so trees small enough get a variant that keeps few registers
// per thread and moves K and V in the same CTA.
#include "common.cuh"

namespace falcon {
namespace {

constexpr int kCompactThreads = 256;
constexpr int kMaxChunksPerThread = 16;  // 128 rows x 32 chunks (D = 256) / 256 threads
constexpr int kSmallChunksPerThread = 4; // the small variant: trees of up to 1024 chunks per matrix
constexpr int kMidChunksPerThread = 6;   // up to 1536 chunks per matrix (96 nodes at head_dim 128)

struct CompactParams {
  int32_t batch, n_layers, n_kv_heads, head_dim, s_cap, path_stride;
  int64_t stride_b, stride_h, stride_s;
  const int32_t* node_off;
  const int32_t* prefix_len;
  int32_t* status;
  void* const* k_layers;
  void* const* v_layers;
  const void* const* k_tree_layers;
  const void* const* v_tree_layers;
  const int32_t* path;
  const int32_t* n_path;
  int32_t* new_len;
  // accepted tokens and features (optional: features == nullptr means none)
  const int32_t* token;
  const __nv_bfloat16* features;
  __nv_bfloat16* features_out;
  int32_t* tokens_out;
  int64_t feat_stride;
  int32_t hidden, out_rows;
  int32_t gather_z;  // the grid's z slice that does the gather in a combined launch
};

// Accepted tokens and features of sequence b: an out-of-place row gather along the path (Section
// 3.4: the accepted tokens and their features are kept for the next drafting phase).  The `n_parts` CTAs of a
// sequence share the 16-byte chunks; the path has been validated into s_path by the caller.
__device__ __forceinline__ void gather_features(const CompactParams& p, int b, int base, int n, const int* s_path,
                                                int part, int n_parts, int tid) {
  const int cpr = p.hidden >> 3;
  const int total = n * cpr;
  for (int idx = part * kCompactThreads + tid; idx < total; idx += n_parts * kCompactThreads) {
    const int j = idx / cpr, c = idx - j * cpr;
    const uint4 x = *reinterpret_cast<const uint4*>(p.features + static_cast<int64_t>(base + s_path[j]) * p.feat_stride + 8 * c);
    *reinterpret_cast<uint4*>(p.features_out + (static_cast<int64_t>(b) * p.out_rows + j) * p.hidden + 8 * c) = x;
  }
  if (part == 0 && tid < n) p.tokens_out[static_cast<int64_t>(b) * p.out_rows + tid] = p.token[base + s_path[tid]];
}

// kBoth: blockIdx.z is the layer and the CTA moves K then V (both held in registers at once);
// otherwise blockIdx.z is 2 * layer + (0 for K, 1 for V).
template <int kChunks, bool kBoth>
__global__ void __launch_bounds__(kCompactThreads) kv_compact_kernel(const CompactParams p) {
  __shared__ int s_path[FALCON_T_MAX];
  __shared__ int s_bad;
  // Under programmatic dependent launch the grid may start while the previous kernel of the stream
  // drains: nothing is read or written before that kernel has completed.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int h = blockIdx.x, b = blockIdx.y;
  const bool gather_slice = p.features != nullptr && static_cast<int>(blockIdx.z) == p.gather_z;
  const int layer = gather_slice ? 0 : (kBoth ? blockIdx.z : (blockIdx.z >> 1));
  const int tid = threadIdx.x;
  constexpr int kMats = kBoth ? 2 : 1;

  const int base = p.node_off[b];
  const int T = p.node_off[b + 1] - base;
  const int L = p.prefix_len[b];
  const int n = p.n_path[b];
  const bool separate = (p.k_tree_layers != nullptr);
  int fault = 0;
  if (T < 1 || T > FALCON_T_MAX || n < 1 || n > T) fault |= FALCON_DEV_BAD_PATH;
  if (!gather_slice) {
    if (L < 0 || L + (separate ? n : T) > p.s_cap) fault |= FALCON_DEV_CAPACITY;
    // the variant was picked from the caller's max_tree: a longer path than it can hold is refused
    if (n > 0 && static_cast<int64_t>(n) * (p.head_dim >> 3) > static_cast<int64_t>(kChunks) * kCompactThreads)
      fault |= FALCON_DEV_CAPACITY;
  } else if (n > p.out_rows) {
    fault |= FALCON_DEV_CAPACITY;
  }
  if (tid == 0) s_bad = 0;
  __syncthreads();
  if (!fault && tid < n) {
    const int t = p.path[static_cast<int64_t>(b) * p.path_stride + tid];
    s_path[tid] = t;
    if (t < 0 || t >= T) s_bad = 1;
  }
  __syncthreads();
  if (s_bad) fault |= FALCON_DEV_BAD_PATH;
  if (gather_slice) {
    if (fault) {
      if (h == 0 && tid == 0) dev_status_or(p.status, b, fault);
      return;
    }
    gather_features(p, b, base, n, s_path, h, gridDim.x, tid);
    return;
  }
  const bool first = (h == 0 && blockIdx.z == 0 && tid == 0);  // one writer of the new length per sequence
  if (fault) {  // leave the cache alone, report, keep the old length
    if (first) {
      dev_status_or(p.status, b, fault);
      p.new_len[b] = L;
    }
    return;
  }
  if (first) p.new_len[b] = L + n;

  __nv_bfloat16* cache[kMats];
  const __nv_bfloat16* tree[kMats];
#pragma unroll
  for (int m = 0; m < kMats; ++m) {
    const bool is_v = kBoth ? (m == 1) : ((blockIdx.z & 1) != 0);
    cache[m] = static_cast<__nv_bfloat16*>(is_v ? p.v_layers[layer] : p.k_layers[layer]) + b * p.stride_b + h * p.stride_h;
    tree[m] = separate ? static_cast<const __nv_bfloat16*>(is_v ? p.v_tree_layers[layer] : p.k_tree_layers[layer])
                       : nullptr;
  }

  const int cpr = p.head_dim >> 3;  // 16-byte chunks per row
  const int total = n * cpr;
  uint4 regs[kMats][kChunks];
#pragma unroll
  for (int m = 0; m < kMats; ++m) {
#pragma unroll
    for (int k = 0; k < kChunks; ++k) {
      const int idx = tid + k * kCompactThreads;
      if (idx < total) {
        const int j = idx / cpr, c = idx - j * cpr;
        const __nv_bfloat16* src =
            separate ? tree[m] + (static_cast<int64_t>(base + s_path[j]) * p.n_kv_heads + h) * p.head_dim
                     : cache[m] + static_cast<int64_t>(L + s_path[j]) * p.stride_s;
        regs[m][k] = *reinterpret_cast<const uint4*>(src + 8 * c);
      }
    }
  }
  __syncthreads();  // every source row is in registers before any destination row is written
#pragma unroll
  for (int m = 0; m < kMats; ++m) {
#pragma unroll
    for (int k = 0; k < kChunks; ++k) {
      const int idx = tid + k * kCompactThreads;
      if (idx < total) {
        const int j = idx / cpr, c = idx - j * cpr;
        *reinterpret_cast<uint4*>(cache[m] + static_cast<int64_t>(L + j) * p.stride_s + 8 * c) = regs[m][k];
      }
    }
  }
}

// The gather alone: grid (parts, B).
__global__ void __launch_bounds__(kCompactThreads) feature_gather_kernel(const CompactParams p) {
  __shared__ int s_path[FALCON_T_MAX];
  __shared__ int s_bad;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int b = blockIdx.y, tid = threadIdx.x;
  const int base = p.node_off[b];
  const int T = p.node_off[b + 1] - base;
  const int n = p.n_path[b];
  int fault = 0;
  if (T < 1 || T > FALCON_T_MAX || n < 1 || n > T) fault |= FALCON_DEV_BAD_PATH;
  if (n > p.out_rows) fault |= FALCON_DEV_CAPACITY;
  if (tid == 0) s_bad = 0;
  __syncthreads();
  if (!fault && tid < n) {
    const int t = p.path[static_cast<int64_t>(b) * p.path_stride + tid];
    s_path[tid] = t;
    if (t < 0 || t >= T) s_bad = 1;
  }
  __syncthreads();
  if (s_bad) fault |= FALCON_DEV_BAD_PATH;
  if (fault) {
    if (blockIdx.x == 0 && tid == 0) dev_status_or(p.status, b, fault);
    return;
  }
  gather_features(p, b, base, n, s_path, blockIdx.x, gridDim.x, tid);
}

void set_gather(CompactParams& p, const falcon_gather_args& g, const int32_t* token) {
  p.token = token;
  p.features = static_cast<const __nv_bfloat16*>(g.features);
  p.features_out = static_cast<__nv_bfloat16*>(g.features_out);
  p.tokens_out = g.tokens_out;
  p.feat_stride = g.feat_stride;
  p.hidden = g.hidden;
  p.out_rows = g.out_rows;
}

}  // namespace

int check_gather_args(const falcon_gather_args& g, int max_tree) {
  if (!g.features || !g.features_out || !g.tokens_out) return FALCON_ERR_INVALID_ARG;
  if (g.hidden < 8 || (g.hidden & 7) || g.feat_stride < g.hidden || (g.feat_stride & 7)) return FALCON_ERR_INVALID_ARG;
  if (g.out_rows < max_tree) return FALCON_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(g.features) | reinterpret_cast<uintptr_t>(g.features_out)) & 15) return FALCON_ERR_INVALID_ARG;
  return FALCON_OK;
}

int launch_feature_gather(falcon_ctx* ctx, const falcon_gather_args& a, cudaStream_t s) {
  if (a.tree.batch > 65535) return FALCON_ERR_CAPACITY;
  CompactParams p = {};
  p.batch = a.tree.batch;
  p.path_stride = a.path_stride;
  p.node_off = a.tree.node_off;
  p.status = a.tree.status;
  p.path = a.path;
  p.n_path = a.n_path;
  set_gather(p, a, a.tree.token);
  const int64_t chunks = static_cast<int64_t>(a.tree.max_tree) * (a.hidden >> 3);
  int parts = static_cast<int>((chunks + 2 * kCompactThreads - 1) / (2 * kCompactThreads));
  if (parts < 1) parts = 1;
  if (parts > 32) parts = 32;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(parts, a.tree.batch);
  cfg.blockDim = dim3(kCompactThreads);
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, feature_gather_kernel, p);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "feature_gather_kernel launch");
  return FALCON_OK;
}

int launch_kv_compact(falcon_ctx* ctx, const falcon_compact_args& a, cudaStream_t s) {
  if (a.tree.batch > 65535 || 2 * static_cast<int64_t>(a.n_layers) + 1 > 65535) return FALCON_ERR_CAPACITY;
  CompactParams p = {};
  p.batch = a.tree.batch;
  p.n_layers = a.n_layers;
  p.n_kv_heads = a.n_kv_heads;
  p.head_dim = a.head_dim;
  p.s_cap = a.s_cap;
  p.path_stride = a.path_stride;
  p.stride_b = a.kv_stride_b;
  p.stride_h = a.kv_stride_h;
  p.stride_s = a.kv_stride_s;
  p.node_off = a.tree.node_off;
  p.prefix_len = a.tree.prefix_len;
  p.status = a.tree.status;
  p.k_layers = a.k_cache_layers;
  p.v_layers = a.v_cache_layers;
  p.k_tree_layers = a.k_tree_layers;
  p.v_tree_layers = a.v_tree_layers;
  p.path = a.path;
  p.n_path = a.n_path;
  p.new_len = a.new_len;
  const int extra = a.gather ? 1 : 0;  // one more z slice of CTAs records the accepted tokens and features
  if (a.gather) set_gather(p, *a.gather, a.tree.token);
  // the path is at most max_tree rows long: small trees take the variant with K and V in one CTA
  const int64_t max_chunks = static_cast<int64_t>(a.tree.max_tree) * (a.head_dim >> 3);
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kCompactThreads);
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  cudaError_t e;
  if (max_chunks <= static_cast<int64_t>(kSmallChunksPerThread) * kCompactThreads) {
    p.gather_z = a.n_layers;
    cfg.gridDim = dim3(a.n_kv_heads, a.tree.batch, a.n_layers + extra);
    e = cudaLaunchKernelEx(&cfg, kv_compact_kernel<kSmallChunksPerThread, true>, p);
  } else if (max_chunks <= static_cast<int64_t>(kMidChunksPerThread) * kCompactThreads) {
    p.gather_z = a.n_layers;
    cfg.gridDim = dim3(a.n_kv_heads, a.tree.batch, a.n_layers + extra);
    e = cudaLaunchKernelEx(&cfg, kv_compact_kernel<kMidChunksPerThread, true>, p);
  } else {
    p.gather_z = 2 * a.n_layers;
    cfg.gridDim = dim3(a.n_kv_heads, a.tree.batch, 2 * a.n_layers + extra);
    e = cudaLaunchKernelEx(&cfg, kv_compact_kernel<kMaxChunksPerThread, false>, p);
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, "kv_compact_kernel launch");
  return FALCON_OK;
}

}  // namespace falcon
