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
  // non-greedy only
  float inv_t_log2e;       // log2(e) / temperature
  const float* uniforms;   // [N]
  float* part_sum;         // [N, chunks] sum of exp((x - chunk max) / temperature)
  int* row_tickets;        // [N]
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

// The longest accepted path of sequence b from the nodes' argmax tokens: thread tid < T brings
// g = the argmax of node tid; every thread of the CTA calls this.
__device__ __forceinline__ void search_tree(const AcceptParams& p, int b, int base, int T_real, int g, int* s_par, int* s_tok,
                                            int* s_g, int* s_key) {
  const int tid = threadIdx.x;
  const int T = min(T_real, FALCON_T_MAX);
  bool bad = (T_real > FALCON_T_MAX);
  if (tid < T) {
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
  }
}


__global__ void __launch_bounds__(kAcceptThreads) tree_accept_kernel(const AcceptParams p) {
  __shared__ Best warp_best[kAcceptThreads / 32];
  __shared__ int s_flag;
  __shared__ int s_par[FALCON_T_MAX], s_tok[FALCON_T_MAX], s_g[FALCON_T_MAX];
  __shared__ int s_key[kAcceptThreads / 32];

  // Under programmatic dependent launch the grid may start while the previous kernel of the stream
  // drains: nothing is read or written before that kernel has completed.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int row = blockIdx.y, chunk = blockIdx.x, tid = threadIdx.x;
  const int c0 = chunk * p.chunk_len;
  const int c1 = min(p.vocab, c0 + p.chunk_len);
  const float* rowp = p.logits + static_cast<int64_t>(row) * p.logits_stride;

  // sequence that owns this row (looked up first: its loads overlap the scan below)
  int lo = 0, hi = p.batch;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (p.node_off[mid] <= row) lo = mid; else hi = mid;
  }
  const int b = lo;
  const int base = p.node_off[b];
  const int T_real = p.node_off[b + 1] - base;
  const int T = min(T_real, FALCON_T_MAX);

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
  int g = 0;
  if (tid < T) {
    Best r{-INFINITY, kNone};
    const int64_t o = static_cast<int64_t>(base + tid) * p.chunks;
    for (int c0f = 0; c0f < p.chunks; c0f += 8) {  // eight partials in flight: the loads are independent
      float v[8];
      int ix[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const bool in = c0f + k < p.chunks;
        v[k] = in ? __ldcg(p.part_val + o + c0f + k) : -INFINITY;
        ix[k] = in ? __ldcg(p.part_idx + o + c0f + k) : kNone;
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) r = merge(r, Best{v[k], ix[k]});
    }
    g = (r.i == kNone) ? 0 : r.i;
    p.argmax_out[base + tid] = g;
  }
  search_tree(p, b, base, T_real, g, s_par, s_tok, s_g, s_key);
  if (tid == 0) p.tickets[b] = 0;  // ready for the next call
}

// The search alone, for callers that already have g (falcon_lm_head_argmax writes it): one CTA per
// sequence.
__global__ void __launch_bounds__(kAcceptThreads) tree_search_kernel(const AcceptParams p) {
  __shared__ int s_par[FALCON_T_MAX], s_tok[FALCON_T_MAX], s_g[FALCON_T_MAX];
  __shared__ int s_key[kAcceptThreads / 32];
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int b = blockIdx.x, tid = threadIdx.x;
  const int base = p.node_off[b];
  const int T_real = p.node_off[b + 1] - base;
  const int g = tid < min(T_real, FALCON_T_MAX) ? p.argmax_out[base + tid] : 0;
  search_tree(p, b, base, T_real, g, s_par, s_tok, s_g, s_key);
}

// ---------------------------------------------------------------------------------------------
// Non-greedy acceptance: g[i] is the target's own draw from softmax(logits[i] / temperature)
// (Section 3.1: the next token is sampled from the LM head's distribution) by the inverse-CDF rule
// with the caller's uniform u[i]: the lowest v whose partial sum of weights exceeds u[i] times the
// total.  One launch.  Every CTA takes one chunk (at most 4096 entries, in registers) of one row:
// chunk maximum, then the chunk's sum of weights relative to it.  The last CTA of a row to finish
// (counter) rescales the chunks' sums to the row maximum, finds the chunk in which the partial sums
// pass the target, loads that chunk again (L2) and finds the position: warp by warp, then row of
// 32 by row, then by a scan over the lanes.  The last row of a sequence (second counter) runs the
// same path search as the greedy call.  fp32 sums: a draw within rounding of a boundary between
// two tokens may fall on either side.
constexpr int kSamplePerLane = 16;
constexpr int kSampleChunkMax = (kAcceptThreads / 32) * 32 * kSamplePerLane;  // 4096

__device__ __forceinline__ float warp_add(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__global__ void __launch_bounds__(kAcceptThreads) tree_sample_kernel(const AcceptParams p) {
  constexpr int kWarps = kAcceptThreads / 32;
  __shared__ Best warp_best[kWarps];
  __shared__ float s_wsum[kWarps];
  __shared__ float s_scaled[64];
  __shared__ float s_bcast[4];
  __shared__ int s_ibcast[4];
  __shared__ int s_flag;
  __shared__ int s_par[FALCON_T_MAX], s_tok[FALCON_T_MAX], s_g[FALCON_T_MAX];
  __shared__ int s_key[kWarps];

  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int row = blockIdx.y, chunk = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const float* rowp = p.logits + static_cast<int64_t>(row) * p.logits_stride;
  int lo = 0, hi = p.batch;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (p.node_off[mid] <= row) lo = mid; else hi = mid;
  }
  const int b = lo;
  const int base = p.node_off[b];
  const int T_real = p.node_off[b + 1] - base;
  const float kq = p.inv_t_log2e;

  // entry k of lane l of warp w is element w * 512 + k * 32 + l of the chunk (coalesced rows of 32)
  auto load_chunk = [&](int ch, float (&x)[kSamplePerLane], bool streaming) {
    const int c0 = ch * p.chunk_len;
    const int n = min(p.vocab, c0 + p.chunk_len) - c0;
#pragma unroll
    for (int k = 0; k < kSamplePerLane; ++k) {
      const int j = warp * (32 * kSamplePerLane) + k * 32 + lane;
      x[k] = j < n ? (streaming ? __ldcs(rowp + c0 + j) : __ldcg(rowp + c0 + j)) : __int_as_float(0x7fc00000);  // NaN = no entry
    }
    return c0;
  };

  // ---- every CTA: the chunk's maximum (and where it first occurs) and its sum of weights ----
  {
    float x[kSamplePerLane];
    const int c0 = load_chunk(chunk, x, true);
    Best mine{-INFINITY, kNone};
#pragma unroll
    for (int k = 0; k < kSamplePerLane; ++k) take(mine, x[k], c0 + warp * (32 * kSamplePerLane) + k * 32 + lane);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      Best other{__shfl_xor_sync(0xffffffffu, mine.v, o), __shfl_xor_sync(0xffffffffu, mine.i, o)};
      mine = merge(mine, other);
    }
    if (lane == 0) warp_best[warp] = mine;
    __syncthreads();
    Best r = warp_best[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) r = merge(r, warp_best[w]);
    float s = 0.f;
    if (r.v > -INFINITY && r.v < INFINITY) {
#pragma unroll
      for (int k = 0; k < kSamplePerLane; ++k)
        if (x[k] == x[k]) s += exp2f((x[k] - r.v) * kq);
    }
    s = warp_add(s);
    if (lane == 0) s_wsum[warp] = s;
    __syncthreads();
    if (tid == 0) {
      float tot = 0.f;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) tot += s_wsum[w];
      const int64_t o = static_cast<int64_t>(row) * p.chunks + chunk;
      p.part_val[o] = r.v;
      p.part_sum[o] = tot;
      p.part_idx[o] = r.i;
      __threadfence();
      s_flag = (atomicAdd(&p.row_tickets[row], 1) == p.chunks - 1);
    }
    __syncthreads();
    if (!s_flag) return;
    __threadfence();
  }

  // ---- last CTA of the row: the chunk in which the partial sums pass u * total ----
  if (tid == 0) {
    const int64_t o = static_cast<int64_t>(row) * p.chunks;
    float M = -INFINITY;
    for (int c = 0; c < p.chunks; ++c) M = fmaxf(M, __ldcg(p.part_val + o + c));
    int direct = -1, cstar = 0;
    float resid = 0.f;
    if (!(M > -INFINITY)) {
      direct = 0;  // nothing to draw from
    } else if (!(M < INFINITY)) {
      for (int c = 0; c < p.chunks && direct < 0; ++c)  // a +inf logit takes everything: its first position
        if (__ldcg(p.part_val + o + c) == M) direct = __ldcg(p.part_idx + o + c);
    } else {
      float total = 0.f;
      for (int c = 0; c < p.chunks; ++c) {
        const float mc = __ldcg(p.part_val + o + c);
        const float sc = mc > -INFINITY ? __ldcg(p.part_sum + o + c) * exp2f((mc - M) * kq) : 0.f;
        s_scaled[c] = sc;
        total += sc;
      }
      const float target = p.uniforms[row] * total;
      float run = 0.f;
      int last = 0;
      cstar = -1;
      for (int c = 0; c < p.chunks; ++c) {
        const float sc = s_scaled[c];
        if (sc > 0.f) last = c;
        if (run + sc > target) {
          cstar = c;
          break;
        }
        run += sc;
      }
      if (cstar < 0) {  // rounding left the target at or past the total: the end of the last chunk that has weight
        cstar = last;
        run -= s_scaled[last];
      }
      resid = target - run;
    }
    s_ibcast[0] = direct;
    s_ibcast[1] = cstar;
    s_bcast[0] = resid;
    s_bcast[1] = M;
    p.row_tickets[row] = 0;  // ready for the next call
  }
  __syncthreads();
  int g = s_ibcast[0];
  if (g < 0) {
    // ---- the position inside that chunk: warp, then row of 32, then lane ----
    const int cstar = s_ibcast[1];
    const float M = s_bcast[1];
    float x[kSamplePerLane], w[kSamplePerLane];
    const int c0 = load_chunk(cstar, x, false);
    float ws = 0.f;
#pragma unroll
    for (int k = 0; k < kSamplePerLane; ++k) {
      w[k] = (x[k] == x[k]) ? exp2f((x[k] - M) * kq) : 0.f;
      ws += w[k];
    }
    ws = warp_add(ws);
    if (lane == 0) s_wsum[warp] = ws;
    __syncthreads();
    // every thread: which warp (the sums are the same in all of them)
    float resid = s_bcast[0], tot = 0.f;
#pragma unroll
    for (int i = 0; i < kWarps; ++i) tot += s_wsum[i];
    resid = fminf(resid, tot * 0.99999f);  // recomputed with the row maximum the chunk may sum to a hair less
    int wstar = -1, wlast = 0;
    float run = 0.f;
#pragma unroll
    for (int i = 0; i < kWarps; ++i) {
      const float v = s_wsum[i];
      if (v > 0.f) wlast = i;
      if (wstar < 0) {
        if (run + v > resid) wstar = i; else run += v;
      }
    }
    if (wstar < 0) {
      wstar = wlast;
      run -= s_wsum[wlast];
    }
    if (warp == wstar) {
      float rw = fminf(resid - run, s_wsum[wstar] * 0.99999f);
      int kstar = -1, klast = 0;
      float wk = 0.f, before = 0.f, acc = 0.f;
#pragma unroll
      for (int k = 0; k < kSamplePerLane; ++k) {
        const float rs = warp_add(w[k]);
        if (rs > 0.f) klast = k;
        if (kstar < 0) {
          if (acc + rs > rw) {
            kstar = k;
            before = acc;
          } else {
            acc += rs;
          }
        }
      }
      if (kstar < 0) kstar = klast;
#pragma unroll
      for (int k = 0; k < kSamplePerLane; ++k)
        if (k == kstar) wk = w[k];
      const float rsel = warp_add(wk);  // (if no row passed the target, `before` is 0 and the clamp below ends the search
                                        // at the last entry of the last row that has weight)
      float incl = wk;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const float t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      const float rl = fminf(rw - before, rsel * 0.99999f);
      const unsigned pass = __ballot_sync(0xffffffffu, wk > 0.f && incl > rl);
      const unsigned any = __ballot_sync(0xffffffffu, wk > 0.f);
      const int lstar = pass ? __ffs(static_cast<int>(pass)) - 1 : (any ? 31 - __clz(static_cast<int>(any)) : 0);
      if (lane == 0) s_ibcast[2] = c0 + wstar * (32 * kSamplePerLane) + kstar * 32 + lstar;
    }
    __syncthreads();
    g = s_ibcast[2];
  }
  if (tid == 0) {
    p.argmax_out[row] = g;
    __threadfence();
    s_flag = (atomicAdd(&p.tickets[b], 1) == T_real - 1);
  }
  __syncthreads();
  if (!s_flag) return;
  __threadfence();
  // ---- last row of sequence b: the path search on the drawn tokens ----
  const int gt = tid < min(T_real, FALCON_T_MAX) ? __ldcg(p.argmax_out + base + tid) : 0;
  search_tree(p, b, base, T_real, gt, s_par, s_tok, s_g, s_key);
  if (tid == 0) p.tickets[b] = 0;  // ready for the next call
}

constexpr int kAcceptMaxChunks = 64;  // vocabulary chunks per row at most (the static scratch is sized by it)

// How a launch splits the vocabulary: enough CTAs for a few waves, chunks of at least 2048 elements
// and a multiple of 4.  Shared by the two entry points so that they cannot drift apart.
void accept_plan(int sm_count, int n_nodes, int vocab, int* chunks_out, int* chunk_len_out) {
  int chunks = (4 * sm_count + n_nodes - 1) / n_nodes;
  const int max_chunks = (vocab + 2047) / 2048;
  if (chunks > max_chunks) chunks = max_chunks;
  if (chunks > kAcceptMaxChunks) chunks = kAcceptMaxChunks;
  if (chunks < 1) chunks = 1;
  int chunk_len = (vocab + chunks - 1) / chunks;
  chunk_len = (chunk_len + 3) & ~3;
  *chunks_out = (vocab + chunk_len - 1) / chunk_len;
  *chunk_len_out = chunk_len;
}

// Kernel parameters from the caller's arguments, the plan and the scratch: `part` holds
// n_nodes * chunks values followed by as many indices, `tickets` one counter per sequence.
AcceptParams accept_params(const falcon_accept_args& a, int chunks, int chunk_len, void* part, int* tickets) {
  AcceptParams p;
  p.batch = a.tree.batch;
  p.total_nodes = a.tree.total_nodes;
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
  p.part_val = static_cast<float*>(part);
  p.part_idx = reinterpret_cast<int32_t*>(part) + static_cast<size_t>(a.tree.total_nodes) * chunks;
  p.tickets = tickets;
  p.inv_t_log2e = 0.f;
  p.uniforms = nullptr;
  p.part_sum = nullptr;
  p.row_tickets = nullptr;
  return p;
}

}  // namespace

int launch_tree_accept(falcon_ctx* ctx, const falcon_accept_args& a, cudaStream_t s) {
  const int N = a.tree.total_nodes;
  if (N > 65535) return FALCON_ERR_CAPACITY;
  int chunks, chunk_len;
  accept_plan(ctx->sm_count, N, a.vocab, &chunks, &chunk_len);

  const size_t part = static_cast<size_t>(N) * chunks;
  int rc = ensure_workspace(ctx, part * 8 + 256);
  if (rc) return rc;
  rc = ensure_tickets(ctx, a.tree.batch, s);
  if (rc) return rc;
  const AcceptParams p = accept_params(a, chunks, chunk_len, ctx->ws, ctx->tickets);

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(chunks, N);
  cfg.blockDim = dim3(kAcceptThreads);
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, tree_accept_kernel, p);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "tree_accept_kernel launch");
  return FALCON_OK;
}

// temperature > 0: the nodes' tokens are drawn instead of taken at the maximum.
int launch_tree_sample(falcon_ctx* ctx, const falcon_accept_args& a, cudaStream_t s) {
  const int N = a.tree.total_nodes, B = a.tree.batch;
  if (N > 65535) return FALCON_ERR_CAPACITY;
  int chunks, chunk_len;
  accept_plan(ctx->sm_count, N, a.vocab, &chunks, &chunk_len);
  const int min_chunks = (a.vocab + kSampleChunkMax - 1) / kSampleChunkMax;  // a chunk is held in registers
  if (chunks < min_chunks) chunks = min_chunks;
  if (chunks > kAcceptMaxChunks) return FALCON_ERR_CAPACITY;
  chunk_len = ((a.vocab + chunks - 1) / chunks + 3) & ~3;
  chunks = (a.vocab + chunk_len - 1) / chunk_len;

  const size_t part = static_cast<size_t>(N) * chunks;
  int rc = ensure_workspace(ctx, part * 12 + 256);
  if (rc) return rc;
  rc = ensure_tickets(ctx, static_cast<size_t>(B) + N, s);
  if (rc) return rc;
  AcceptParams p = accept_params(a, chunks, chunk_len, ctx->ws, ctx->tickets);
  p.part_sum = reinterpret_cast<float*>(p.part_idx + part);
  p.row_tickets = ctx->tickets + B;
  p.uniforms = a.uniforms;
  p.inv_t_log2e = kLog2e / a.temperature;

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(chunks, N);
  cfg.blockDim = dim3(kAcceptThreads);
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, tree_sample_kernel, p);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "tree_sample_kernel launch");
  return FALCON_OK;
}

// The nodes' argmax tokens are already in a.argmax_out (written by an earlier call on the stream):
// the path search alone, one CTA per sequence.
int launch_tree_search(falcon_ctx* ctx, const falcon_accept_args& a, cudaStream_t s) {
  const AcceptParams p = accept_params(a, 1, 4, nullptr, nullptr);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(a.tree.batch);
  cfg.blockDim = dim3(kAcceptThreads);
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, tree_search_kernel, p);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "tree_search_kernel launch");
  return FALCON_OK;
}

}  // namespace falcon

// ---------------------------------------------------------------------------------------------
// falcon_tree_accept_static: the same acceptance kernel for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at all: an inference server whose device
// memory is handed out entirely by its own pool, a process running under a fixed memory budget
// (an MPS client with a memory limit, a container whose quota is already committed), or a decode
// loop that cannot tolerate the implicit synchronisation an allocation may bring.  For them the
// scratch of the acceptance kernel (the per-chunk argmax partials and the arrival counters) lives
// in the fixed array below, which is part of the library image: every GPU that loads the library
// holds these bytes until the process exits, whether or not this entry point is ever called.
// ---------------------------------------------------------------------------------------------
#include <mutex>

namespace falcon {
namespace {

constexpr int kStaticMaxNodes = FALCON_STATIC_MAX_NODES;
constexpr int kStaticMaxBatch = FALCON_STATIC_MAX_BATCH;
constexpr int kStaticMaxChunks = kAcceptMaxChunks;
constexpr size_t kStaticPartBytes = static_cast<size_t>(kStaticMaxNodes) * kStaticMaxChunks * 8;  // values + indices
constexpr size_t kStaticBytes = kStaticPartBytes + static_cast<size_t>(kStaticMaxBatch) * sizeof(int);

// In host code this name is only a handle for cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) unsigned char g_accept_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
struct StaticSlot {
  void* ptr = nullptr;  // device address of g_accept_scratch on this device
  int sm_count = 0;
};
StaticSlot g_slots[kMaxDevices];
std::mutex g_slots_mutex;

// Once per device, with that device current: resolve the array's device address.
int static_scratch(int device, StaticSlot* out) {
  std::lock_guard<std::mutex> lock(g_slots_mutex);
  StaticSlot& slot = g_slots[device];
  if (slot.ptr == nullptr) {
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_accept_scratch);
    if (e != cudaSuccess || ptr == nullptr) return FALCON_ERR_CUDA;
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess || sms < 1) return FALCON_ERR_CUDA;
    slot.sm_count = sms;
    slot.ptr = ptr;
  }
  *out = slot;
  return FALCON_OK;
}

}  // namespace
}  // namespace falcon

extern "C" int falcon_tree_accept_static(const falcon_accept_args* a, void* stream) {
  using namespace falcon;
  if (!a) return FALCON_ERR_INVALID_ARG;
  int rc = check_tree_desc(a->tree, true);
  if (rc) return rc;
  if (!a->logits || !a->argmax_out || !a->path || !a->n_path || !a->next_token) return FALCON_ERR_INVALID_ARG;
  if (a->vocab < 1 || a->logits_stride < a->vocab) return FALCON_ERR_INVALID_ARG;
  if (a->path_stride < a->tree.max_tree) return FALCON_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(a->logits) & 3) return FALCON_ERR_INVALID_ARG;
  if (a->temperature != 0.f) return FALCON_ERR_UNSUPPORTED;  // the fixed scratch is sized for the greedy call
  // sizes beyond the fixed scratch are refused, never truncated
  if (a->tree.total_nodes > kStaticMaxNodes || a->tree.batch > kStaticMaxBatch) return FALCON_ERR_CAPACITY;

  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return FALCON_ERR_CUDA;
  StaticSlot slot;
  rc = static_scratch(device, &slot);
  if (rc) return rc;

  const int N = a->tree.total_nodes;
  int chunks, chunk_len;
  accept_plan(slot.sm_count, N, a->vocab, &chunks, &chunk_len);

  unsigned char* base = static_cast<unsigned char*>(slot.ptr);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // The array keeps whatever the previous call left.  The partials are fully rewritten by this
  // launch; the arrival counters must start at zero, so they are cleared on the stream first.
  cudaError_t e = cudaMemsetAsync(base + kStaticPartBytes, 0, static_cast<size_t>(a->tree.batch) * sizeof(int), s);
  if (e != cudaSuccess) return FALCON_ERR_CUDA;
  const AcceptParams p = accept_params(*a, chunks, chunk_len, base, reinterpret_cast<int*>(base + kStaticPartBytes));
  dim3 grid(chunks, N);
  tree_accept_kernel<<<grid, kAcceptThreads, 0, s>>>(p);
  e = cudaGetLastError();
  return e == cudaSuccess ? FALCON_OK : FALCON_ERR_CUDA;
}
