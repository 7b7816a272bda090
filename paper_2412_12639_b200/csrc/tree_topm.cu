// falcon_topm: the m best entries of every logits row, best first (the children a tree
// node gets when the decoding tree is grown, Appendix A).
//
// Order: larger value first, the lower index among equal values; a NaN counts as -inf.
// One launch.  Grid (chunks, rows): a CTA keeps its vocabulary chunk in shared memory and
// takes the chunk's m best in m rounds of a block-wide (value, index) maximum, striking each
// winner out; the last CTA of a row to finish (arrival counter) runs the same m rounds over
// the chunks' candidates and writes the row's result.  The row is read from HBM once
// (4 V bytes); everything after that is shared memory and a few hundred bytes of scratch.
#include "common.cuh"

namespace falcon {
namespace {

constexpr int kTopmThreads = 256;
constexpr int kTopmChunkMax = 4096;               // floats of one chunk held in shared memory
constexpr int kTopmCandMax = 64 * FALCON_TOPM_MAX; // candidates of one row in the last CTA

struct TopmParams {
  int32_t n_rows, vocab, m, chunks, chunk_len;
  int64_t logits_stride;
  const float* logits;
  float* top_val;
  int32_t* top_idx;
  float* part_val;    // [rows, chunks, m]
  int32_t* part_idx;  // [rows, chunks, m]
  int32_t* tickets;   // [rows], zero between calls
};

struct Cand {
  float v;
  int i;
};

// a entry that was struck out is NaN in shared memory; live entries never are (NaN inputs are -inf)
__device__ __forceinline__ bool better(float v, int i, const Cand& b) {
  return b.i < 0 || v > b.v || (v == b.v && i < b.i);
}

// Block-wide best of (key[j], id(j)) over j in [0, n), with ties to the lower id.  ids ascend with j
// inside a thread's strided walk only per residue, so the tie rule is applied explicitly everywhere.
template <typename IdFn>
__device__ __forceinline__ Cand block_best(const float* key, int n, IdFn id, Cand* warp_best, int* slot_out) {
  const int tid = threadIdx.x;
  Cand mine{0.f, -1};
  int slot = -1;
  for (int j = tid; j < n; j += kTopmThreads) {
    const float x = key[j];
    if (x == x) {  // not struck out
      const int ix = id(j);
      if (better(x, ix, mine)) {
        mine = Cand{x, ix};
        slot = j;
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, mine.v, o);
    const int oi = __shfl_xor_sync(0xffffffffu, mine.i, o);
    const int os = __shfl_xor_sync(0xffffffffu, slot, o);
    if (oi >= 0 && better(ov, oi, mine)) {
      mine = Cand{ov, oi};
      slot = os;
    }
  }
  __shared__ int warp_slot[kTopmThreads / 32];
  if ((tid & 31) == 0) {
    warp_best[tid >> 5] = mine;
    warp_slot[tid >> 5] = slot;
  }
  __syncthreads();
  Cand r = warp_best[0];
  int rs = warp_slot[0];
#pragma unroll
  for (int w = 1; w < kTopmThreads / 32; ++w) {
    const Cand c = warp_best[w];
    if (c.i >= 0 && better(c.v, c.i, r)) {
      r = c;
      rs = warp_slot[w];
    }
  }
  *slot_out = rs;
  __syncthreads();  // warp_best may be rewritten by the next round
  return r;
}

__global__ void __launch_bounds__(kTopmThreads) tree_topm_kernel(const TopmParams p) {
  __shared__ float s_key[kTopmChunkMax];
  __shared__ int s_idx[kTopmCandMax];
  __shared__ Cand warp_best[kTopmThreads / 32];
  __shared__ int s_last;

  // Under programmatic dependent launch the grid may start while the previous kernel of the stream
  // drains: nothing is read or written before that kernel has completed.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int row = blockIdx.y, chunk = blockIdx.x, tid = threadIdx.x;
  const int c0 = chunk * p.chunk_len;
  const int n = min(p.vocab, c0 + p.chunk_len) - c0;  // >= 1 by construction of the grid
  const float* rowp = p.logits + static_cast<int64_t>(row) * p.logits_stride + c0;

  for (int j = tid; j < n; j += kTopmThreads) {
    const float x = __ldcs(rowp + j);
    s_key[j] = (x == x) ? x : -INFINITY;
  }
  __syncthreads();

  // the chunk's best min(m, n) entries
  const int take = min(p.m, n);
  const int64_t po = (static_cast<int64_t>(row) * p.chunks + chunk) * p.m;
  for (int r = 0; r < p.m; ++r) {
    if (r < take) {
      int slot;
      const Cand c = block_best(s_key, n, [&](int j) { return c0 + j; }, warp_best, &slot);
      if (tid == 0) {
        p.part_val[po + r] = c.v;
        p.part_idx[po + r] = c.i;
        s_key[slot] = __int_as_float(0x7fc00000);  // struck out
      }
      __syncthreads();
    } else if (tid == 0) {
      p.part_val[po + r] = -INFINITY;
      p.part_idx[po + r] = -1;  // no such entry
    }
  }

  if (tid == 0) {
    __threadfence();
    s_last = (atomicAdd(&p.tickets[row], 1) == p.chunks - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();

  // ---- last CTA of the row: the same rounds over the chunks' candidates ----
  const int nc = p.chunks * p.m;
  const int64_t ro = static_cast<int64_t>(row) * nc;
  for (int j = tid; j < nc; j += kTopmThreads) {
    const int ix = __ldcg(p.part_idx + ro + j);
    s_idx[j] = ix;
    s_key[j] = (ix >= 0) ? __ldcg(p.part_val + ro + j) : __int_as_float(0x7fc00000);
  }
  __syncthreads();
  for (int r = 0; r < p.m; ++r) {
    int slot;
    const Cand c = block_best(s_key, nc, [&](int j) { return s_idx[j]; }, warp_best, &slot);
    if (tid == 0) {
      p.top_val[static_cast<int64_t>(row) * p.m + r] = c.v;
      p.top_idx[static_cast<int64_t>(row) * p.m + r] = c.i;
      s_key[slot] = __int_as_float(0x7fc00000);
    }
    __syncthreads();
  }
  if (tid == 0) p.tickets[row] = 0;  // ready for the next call
}

}  // namespace

int launch_tree_topm(falcon_ctx* ctx, const falcon_topm_args& a, cudaStream_t s) {
  const int N = a.n_rows;
  if (N > 65535) return FALCON_ERR_CAPACITY;
  // enough CTAs for a few waves; a chunk holds at least m entries and fits in shared memory
  int chunks = (4 * ctx->sm_count + N - 1) / N;
  const int max_chunks = (a.vocab + 2047) / 2048;
  if (chunks > max_chunks) chunks = max_chunks;
  if (chunks > 64) chunks = 64;
  const int min_chunks = (a.vocab + kTopmChunkMax - 1) / kTopmChunkMax;
  if (chunks < min_chunks) chunks = min_chunks;
  if (chunks > 64) return FALCON_ERR_CAPACITY;  // vocabulary beyond 64 x 4096 entries
  int chunk_len = (a.vocab + chunks - 1) / chunks;
  chunk_len = (chunk_len + 3) & ~3;
  if (chunk_len > kTopmChunkMax) chunk_len = kTopmChunkMax;
  chunks = (a.vocab + chunk_len - 1) / chunk_len;

  const size_t part = static_cast<size_t>(N) * chunks * a.m;
  int rc = ensure_workspace(ctx, part * 8 + 256);
  if (rc) return rc;
  rc = ensure_tickets(ctx, N);
  if (rc) return rc;

  TopmParams p;
  p.n_rows = N;
  p.vocab = a.vocab;
  p.m = a.m;
  p.chunks = chunks;
  p.chunk_len = chunk_len;
  p.logits_stride = a.logits_stride;
  p.logits = a.logits;
  p.top_val = a.top_val;
  p.top_idx = a.top_idx;
  p.part_val = static_cast<float*>(ctx->ws);
  p.part_idx = reinterpret_cast<int32_t*>(static_cast<float*>(ctx->ws) + part);
  p.tickets = ctx->tickets;

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(chunks, N);
  cfg.blockDim = dim3(kTopmThreads);
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, tree_topm_kernel, p);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "tree_topm_kernel launch");
  return FALCON_OK;
}

}  // namespace falcon
