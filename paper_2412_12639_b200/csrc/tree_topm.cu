// falcon_topm: the m best entries of every logits row, best first (the children a tree
// node gets when the decoding tree is grown, Appendix A).
//
// Order: larger value first, the lower index among equal values; a NaN counts as -inf.
// One launch, no block-wide rounds.  Values become 32-bit keys whose unsigned order is the
// float order (key 0 = "no entry"), so that a warp finds its best entry with two redux.sync
// instructions (maximum key, then minimum index among its holders).  Every selection is a warp
// that holds up to 16 entries per lane in registers, each lane's sorted once by a sorting network,
// and takes its m best in m such rounds, the winning lane dropping the head of its list:
//   A  grid (chunks, rows), 8 warps per CTA: each warp loads 512 entries of the CTA's chunk
//      straight into registers and leaves its m best in shared memory;
//   B  warp 0 selects the chunk's m best among those 8 x m and writes them to scratch;
//   C  the last CTA of a row to finish (arrival counter) spreads the chunks' candidates over
//      its 8 warps, m best each;  D  its warp 0 selects the row's result among those.
// The row is read from HBM once (4 V bytes).

#include "common.cuh"

namespace falcon {
namespace {

constexpr int kTopmThreads = 256;
constexpr int kTopmWarps = kTopmThreads / 32;
constexpr int kTopmPerLane = 16;                                  // entries a lane can hold
constexpr int kTopmChunkMax = kTopmWarps * 32 * kTopmPerLane;     // 4096 entries per CTA
constexpr int kTopmCandMax = 64 * FALCON_TOPM_MAX;                // candidates of one row in the last CTA
static_assert(kTopmCandMax <= kTopmChunkMax, "the last CTA holds a row's candidates like a chunk");
static_assert(kTopmWarps * FALCON_TOPM_MAX <= 32 * kTopmPerLane, "one warp holds all warps' candidates");

struct TopmParams {
  int32_t n_rows, vocab, m, chunks, chunk_len;
  int64_t logits_stride;
  const float* logits;
  float* top_val;
  int32_t* top_idx;
  uint32_t* part_key;  // [rows, chunks, m]
  int32_t* part_idx;   // [rows, chunks, m]
  int32_t* tickets;    // [rows], zero between calls
};

// float -> key: unsigned order of the keys = order of the values; NaN -> -inf, -0 -> +0; never 0
__device__ __forceinline__ uint32_t to_key(float x) {
  x = (x == x) ? x + 0.f : -INFINITY;
  const uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float from_key(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// One entry as a 64-bit word whose unsigned order is the selection order: key in the upper half,
// the complemented index in the lower one (so that the lower index is the larger word); 0 = none.
__device__ __forceinline__ uint64_t entry(uint32_t key, int id) {
  return key ? (static_cast<uint64_t>(key) << 32) | static_cast<uint32_t>(~id) : 0ull;
}

// Batcher's odd-even merge sort for 16 inputs (63 compare-exchanges), descending.
__device__ __forceinline__ void sort16_desc(uint64_t (&e)[16]) {
  constexpr int kNet[63][2] = {
      {0, 1},   {2, 3},   {0, 2},   {1, 3},   {1, 2},   {4, 5},   {6, 7},   {4, 6},   {5, 7},   {5, 6},   {0, 4},
      {2, 6},   {2, 4},   {1, 5},   {3, 7},   {3, 5},   {1, 2},   {3, 4},   {5, 6},   {8, 9},   {10, 11}, {8, 10},
      {9, 11},  {9, 10},  {12, 13}, {14, 15}, {12, 14}, {13, 15}, {13, 14}, {8, 12},  {10, 14}, {10, 12}, {9, 13},
      {11, 15}, {11, 13}, {9, 10},  {11, 12}, {13, 14}, {0, 8},   {4, 12},  {4, 8},   {2, 10},  {6, 14},  {6, 10},
      {2, 4},   {6, 8},   {10, 12}, {1, 9},   {5, 13},  {5, 9},   {3, 11},  {7, 15},  {7, 11},  {3, 5},   {7, 9},
      {11, 13}, {1, 2},   {3, 4},   {5, 6},   {7, 8},   {9, 10},  {11, 12}, {13, 14}};
#pragma unroll
  for (int s = 0; s < 63; ++s) {
    const uint64_t x = e[kNet[s][0]], y = e[kNet[s][1]];
    e[kNet[s][0]] = x > y ? x : y;
    e[kNet[s][1]] = x > y ? y : x;
  }
}

// The warp's `rounds` best entries, best first, among the 16 entries each lane holds.  Every lane
// sorts its own entries once; a round is then two redux.sync (the largest key among the lanes'
// heads, the lowest index among its holders) and, in the one lane that held the winner, a shift
// of its list.  emit(round, key, id) is called by every lane (key 0 when nothing is left).
template <typename EmitFn>
__device__ __forceinline__ void warp_rounds(uint64_t (&e)[kTopmPerLane], int rounds, EmitFn emit) {
  static_assert(kTopmPerLane == 16, "the sorting network is for 16 entries");
  sort16_desc(e);
  for (int r = 0; r < rounds; ++r) {
    const uint32_t hk = static_cast<uint32_t>(e[0] >> 32), hn = static_cast<uint32_t>(e[0]);  // head: key, ~index
    const uint32_t kmax = __reduce_max_sync(0xffffffffu, hk);
    const uint32_t nmax = __reduce_max_sync(0xffffffffu, (hk == kmax && kmax != 0u) ? hn : 0u);
    emit(r, kmax, static_cast<int>(~nmax));
    if (kmax != 0u && hk == kmax && hn == nmax) {  // the one lane that held it: drop the head
#pragma unroll
      for (int k = 0; k + 1 < kTopmPerLane; ++k) e[k] = e[k + 1];
      e[kTopmPerLane - 1] = 0ull;
    }
  }
}

__global__ void __launch_bounds__(kTopmThreads) tree_topm_kernel(const TopmParams p) {
  __shared__ uint32_t s_key[kTopmWarps][FALCON_TOPM_MAX];
  __shared__ int s_id[kTopmWarps][FALCON_TOPM_MAX];
  __shared__ int s_last;

  // Under programmatic dependent launch the grid may start while the previous kernel of the stream
  // drains: nothing is read or written before that kernel has completed.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int row = blockIdx.y, chunk = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int c0 = chunk * p.chunk_len;
  const int n = min(p.vocab, c0 + p.chunk_len) - c0;  // >= 1 by construction of the grid
  const float* rowp = p.logits + static_cast<int64_t>(row) * p.logits_stride + c0;
  const int m = p.m;

  // ---- A: each warp's m best of its 512 entries (coalesced 128-byte loads, 16 in flight per lane) ----
  {
    uint64_t e[kTopmPerLane];
#pragma unroll
    for (int k = 0; k < kTopmPerLane; ++k) {
      const int j = warp * (32 * kTopmPerLane) + k * 32 + lane;
      const bool in = j < n;
      e[k] = entry(in ? to_key(__ldcs(rowp + (in ? j : 0))) : 0u, c0 + j);
    }
    warp_rounds(e, m, [&](int r, uint32_t k, int i) {
      if (lane == 0) {
        s_key[warp][r] = k;
        s_id[warp][r] = i;
      }
    });
  }
  __syncthreads();

  // ---- B: warp 0 takes the chunk's m best among the warps' candidates ----
  auto from_shared = [&](uint64_t (&e)[kTopmPerLane]) {
#pragma unroll
    for (int k = 0; k < kTopmPerLane; ++k) {
      const int j = k * 32 + lane;  // candidate j = (warp j % 8, round j / 8)
      const bool in = j < kTopmWarps * m;
      e[k] = in ? entry(s_key[j % kTopmWarps][j / kTopmWarps], s_id[j % kTopmWarps][j / kTopmWarps]) : 0ull;
    }
  };
  if (warp == 0) {
    uint64_t e[kTopmPerLane];
    from_shared(e);
    const int64_t po = (static_cast<int64_t>(row) * p.chunks + chunk) * m;
    warp_rounds(e, m, [&](int r, uint32_t k, int i) {
      if (lane == 0) {
        p.part_key[po + r] = k;  // key 0: the chunk has fewer than m entries
        p.part_idx[po + r] = i;
      }
    });
    if (lane == 0) {
      __threadfence();
      s_last = (atomicAdd(&p.tickets[row], 1) == p.chunks - 1);
    }
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();

  // ---- C: last CTA of the row: the chunks' candidates, spread over the warps ----
  {
    const int nc = p.chunks * m;  // <= kTopmCandMax
    const int64_t ro = static_cast<int64_t>(row) * nc;
    uint64_t e[kTopmPerLane];
#pragma unroll
    for (int k = 0; k < kTopmPerLane; ++k) {
      const int j = warp * (32 * kTopmPerLane) + k * 32 + lane;
      const bool in = j < nc;
      e[k] = in ? entry(__ldcg(p.part_key + ro + j), __ldcg(p.part_idx + ro + j)) : 0ull;
    }
    warp_rounds(e, m, [&](int r, uint32_t k, int i) {
      if (lane == 0) {
        s_key[warp][r] = k;
        s_id[warp][r] = i;
      }
    });
  }
  __syncthreads();

  // ---- D: warp 0 writes the row's result ----
  if (warp == 0) {
    uint64_t e[kTopmPerLane];
    from_shared(e);
    warp_rounds(e, m, [&](int r, uint32_t k, int i) {
      if (lane == 0) {
        p.top_val[static_cast<int64_t>(row) * m + r] = from_key(k);
        p.top_idx[static_cast<int64_t>(row) * m + r] = i;
      }
    });
    if (lane == 0) p.tickets[row] = 0;  // ready for the next call
  }
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
  rc = ensure_tickets(ctx, N, s);
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
  p.part_key = static_cast<uint32_t*>(ctx->ws);
  p.part_idx = reinterpret_cast<int32_t*>(static_cast<uint32_t*>(ctx->ws) + part);
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
