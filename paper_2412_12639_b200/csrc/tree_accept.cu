// falcon_tree_accept: per-node vocabulary argmax and the longest accepted path,
// one launch.  Every CTA scans one chunk of one logits row with 16-byte loads;
// the last CTA to finish a sequence (arrival counter) folds the chunk partials
// into g[] and searches the tree.  HBM-bound: the N*V fp32 logits are read once.
#include <cfloat>
#include <climits>

#include "common.cuh"

namespace falcon {
namespace {

constexpr int kAcceptThreads = 256;
constexpr int kNone = INT_MAX;

struct AcceptParams {
  int32_t batch, total_nodes, vocab, chunks, chunk_len, path_stride;
  int64_t logits_stride;
  const int32_t* node_off;
  const int32_t* parent;
  const int32_t* token;
  int32_t* status;
  const float* logits;
  int32_t* argmax_out;
  int32_t* path;
  int32_t* n_path;
  int32_t* next_token;
  float* part_val;  // [N, chunks]
  int32_t* part_idx;
  int* tickets;     // [B]
};

struct Best {
  float v;
  int i;
};

// Larger value wins; equal values keep the lower index.  (-inf, kNone) is "nothing seen".
__device__ __forceinline__ Best merge(Best a, Best b) {
  if (b.v > a.v || (b.v == a.v && b.i < a.i)) return b;
  return a;
}

__device__ __forceinline__ void take(Best& s, float x, int i) {
  if (x > s.v) {  // strict: within a thread indices ascend, so the first maximum stays; NaN never wins
    s.v = x;
    s.i = i;
  }
}

__global__ void __launch_bounds__(kAcceptThreads) tree_accept_kernel(const AcceptParams p) {
  __shared__ Best warp_best[kAcceptThreads / 32];
  __shared__ int s_flag;
  __shared__ int s_par[FALCON_T_MAX], s_tok[FALCON_T_MAX], s_g[FALCON_T_MAX];
  __shared__ int s_key[kAcceptThreads / 32];

  const int row = blockIdx.y, chunk = blockIdx.x, tid = threadIdx.x;
  const int c0 = chunk * p.chunk_len;
  const int c1 = min(p.vocab, c0 + p.chunk_len);
  const float* rowp = p.logits + static_cast<int64_t>(row) * p.logits_stride;

  Best mine{-INFINITY, kNone};
  if (c0 < c1) {
    // scalar head up to the first 16-byte boundary, float4 body, scalar tail
    const int mis = static_cast<int>((reinterpret_cast<uintptr_t>(rowp + c0) >> 2) & 3);
    const int head = min(c1 - c0, (4 - mis) & 3);
    if (tid < head) take(mine, __ldcs(rowp + c0 + tid), c0 + tid);
    const int b0 = c0 + head;
    const int nvec = (c1 - b0) >> 2;
    const float4* vp = reinterpret_cast<const float4*>(rowp + b0);
#pragma unroll 4
    for (int k = tid; k < nvec; k += kAcceptThreads) {
      const float4 x = __ldcs(vp + k);
      const int i = b0 + 4 * k;
      take(mine, x.x, i);
      take(mine, x.y, i + 1);
      take(mine, x.z, i + 2);
      take(mine, x.w, i + 3);
    }
    const int t0 = b0 + 4 * nvec;
    if (tid < c1 - t0) take(mine, __ldcs(rowp + t0 + tid), t0 + tid);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Best other{__shfl_xor_sync(0xffffffffu, mine.v, o), __shfl_xor_sync(0xffffffffu, mine.i, o)};
    mine = merge(mine, other);
  }
  if ((tid & 31) == 0) warp_best[tid >> 5] = mine;
  __syncthreads();

  // sequence that owns this row
  int lo = 0, hi = p.batch;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (p.node_off[mid] <= row) lo = mid; else hi = mid;
  }
  const int b = lo;
  const int base = p.node_off[b];
  const int T_real = p.node_off[b + 1] - base;
  const int T = min(T_real, FALCON_T_MAX);

  if (tid == 0) {
    Best r = warp_best[0];
#pragma unroll
    for (int w = 1; w < kAcceptThreads / 32; ++w) r = merge(r, warp_best[w]);
    p.part_val[static_cast<int64_t>(row) * p.chunks + chunk] = r.v;
    p.part_idx[static_cast<int64_t>(row) * p.chunks + chunk] = r.i;
    __threadfence();
    const int arrived = atomicAdd(&p.tickets[b], 1);
    s_flag = (arrived == T_real * p.chunks - 1);
  }
  __syncthreads();
  if (!s_flag) return;
  __threadfence();

  // ---- last CTA of sequence b: fold the partials, then search the tree ----
  bool bad = (T_real > FALCON_T_MAX);
  if (tid < T) {
    Best r{-INFINITY, kNone};
    const int64_t o = static_cast<int64_t>(base + tid) * p.chunks;
    for (int c = 0; c < p.chunks; ++c) r = merge(r, Best{__ldcg(p.part_val + o + c), __ldcg(p.part_idx + o + c)});
    const int g = (r.i == kNone) ? 0 : r.i;
    p.argmax_out[base + tid] = g;
    s_g[tid] = g;
    const int pr = p.parent[base + tid];
    s_par[tid] = pr;
    s_tok[tid] = p.token[base + tid];
    bad = bad || ((tid == 0) ? (pr != -1) : (pr < 0 || pr >= tid));
  }
  const int any_bad = __syncthreads_or(bad ? 1 : 0);

  // alive(c): every non-root node on the chain root..c carries the argmax of its parent
  int key = -1;
  if (tid < T && !any_bad) {
    bool alive = true;
    int depth = 0, u = tid;
    while (u != 0 && depth < T) {
      const int pu = s_par[u];
      alive = alive && (s_tok[u] == s_g[pu]);
      u = pu;
      ++depth;
    }
    if (alive) key = depth * 256 + (255 - tid);  // deeper wins, then the lower index
  }
  if (tid == 0 && any_bad) key = 255;  // malformed tree: root only
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) key = max(key, __shfl_xor_sync(0xffffffffu, key, o));
  if ((tid & 31) == 0) s_key[tid >> 5] = key;
  __syncthreads();
  key = s_key[0];
#pragma unroll
  for (int w = 1; w < kAcceptThreads / 32; ++w) key = max(key, s_key[w]);
  const int best = 255 - (key & 255);
  const int n = (key >> 8) + 1;

  int32_t* prow = p.path + static_cast<int64_t>(b) * p.path_stride;
  for (int j = n + tid; j < p.path_stride; j += kAcceptThreads) prow[j] = -1;
  if (tid == 0) {
    int u = best;
    for (int j = n - 1; j >= 0; --j) {
      prow[j] = u;
      u = s_par[u];
    }
    p.n_path[b] = n;
    p.next_token[b] = s_g[best];
    if (any_bad) dev_status_or(p.status, b, FALCON_DEV_BAD_TREE);
    p.tickets[b] = 0;  // ready for the next call
  }
}

}  // namespace

int launch_tree_accept(falcon_ctx* ctx, const falcon_accept_args& a, cudaStream_t s) {
  const int N = a.tree.total_nodes;
  if (N > 65535) return FALCON_ERR_CAPACITY;
  // enough CTAs for a few waves, chunks of at least 2048 elements
  int chunks = (4 * ctx->sm_count + N - 1) / N;
  const int max_chunks = (a.vocab + 2047) / 2048;
  if (chunks > max_chunks) chunks = max_chunks;
  if (chunks > 64) chunks = 64;
  if (chunks < 1) chunks = 1;
  int chunk_len = (a.vocab + chunks - 1) / chunks;
  chunk_len = (chunk_len + 3) & ~3;
  chunks = (a.vocab + chunk_len - 1) / chunk_len;

  const size_t part = static_cast<size_t>(N) * chunks;
  int rc = ensure_workspace(ctx, part * 8 + 256);
  if (rc) return rc;
  rc = ensure_tickets(ctx, a.tree.batch);
  if (rc) return rc;

  AcceptParams p;
  p.batch = a.tree.batch;
  p.total_nodes = N;
  p.vocab = a.vocab;
  p.chunks = chunks;
  p.chunk_len = chunk_len;
  p.path_stride = a.path_stride;
  p.logits_stride = a.logits_stride;
  p.node_off = a.tree.node_off;
  p.parent = a.tree.parent;
  p.token = a.tree.token;
  p.status = a.tree.status;
  p.logits = a.logits;
  p.argmax_out = a.argmax_out;
  p.path = a.path;
  p.n_path = a.n_path;
  p.next_token = a.next_token;
  p.part_val = static_cast<float*>(ctx->ws);
  p.part_idx = reinterpret_cast<int32_t*>(static_cast<float*>(ctx->ws) + part);
  p.tickets = ctx->tickets;

  dim3 grid(chunks, N);
  tree_accept_kernel<<<grid, kAcceptThreads, 0, s>>>(p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "tree_accept_kernel launch");
  return FALCON_OK;
}

}  // namespace falcon
