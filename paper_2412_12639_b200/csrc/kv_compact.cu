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
};

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
  const int layer = kBoth ? blockIdx.z : (blockIdx.z >> 1);
  const int tid = threadIdx.x;
  constexpr int kMats = kBoth ? 2 : 1;

  const int base = p.node_off[b];
  const int T = p.node_off[b + 1] - base;
  const int L = p.prefix_len[b];
  const int n = p.n_path[b];
  const bool separate = (p.k_tree_layers != nullptr);
  int fault = 0;
  if (T < 1 || T > FALCON_T_MAX || n < 1 || n > T) fault |= FALCON_DEV_BAD_PATH;
  if (L < 0 || L + (separate ? n : T) > p.s_cap) fault |= FALCON_DEV_CAPACITY;
  // the variant was picked from the caller's max_tree: a longer path than it can hold is refused
  if (n > 0 && static_cast<int64_t>(n) * (p.head_dim >> 3) > static_cast<int64_t>(kChunks) * kCompactThreads)
    fault |= FALCON_DEV_CAPACITY;
  if (tid == 0) s_bad = 0;
  __syncthreads();
  if (!fault && tid < n) {
    const int t = p.path[static_cast<int64_t>(b) * p.path_stride + tid];
    s_path[tid] = t;
    if (t < 0 || t >= T) s_bad = 1;
  }
  __syncthreads();
  if (s_bad) fault |= FALCON_DEV_BAD_PATH;
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

}  // namespace

int launch_kv_compact(falcon_ctx* ctx, const falcon_compact_args& a, cudaStream_t s) {
  if (a.tree.batch > 65535 || 2 * static_cast<int64_t>(a.n_layers) > 65535) return FALCON_ERR_CAPACITY;
  CompactParams p;
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
    cfg.gridDim = dim3(a.n_kv_heads, a.tree.batch, a.n_layers);
    e = cudaLaunchKernelEx(&cfg, kv_compact_kernel<kSmallChunksPerThread, true>, p);
  } else if (max_chunks <= static_cast<int64_t>(kMidChunksPerThread) * kCompactThreads) {
    cfg.gridDim = dim3(a.n_kv_heads, a.tree.batch, a.n_layers);
    e = cudaLaunchKernelEx(&cfg, kv_compact_kernel<kMidChunksPerThread, true>, p);
  } else {
    cfg.gridDim = dim3(a.n_kv_heads, a.tree.batch, 2 * a.n_layers);
    e = cudaLaunchKernelEx(&cfg, kv_compact_kernel<kMaxChunksPerThread, false>, p);
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, "kv_compact_kernel launch");
  return FALCON_OK;
}

}  // namespace falcon
