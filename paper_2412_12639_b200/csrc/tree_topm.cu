// falcon_topm: the m best entries of every logits row, best first (the children a tree
// node gets when the decoding tree is grown, Appendix A).
//
// Order: larger value first, the lower index among equal values; a NaN counts as -inf.
// One launch, no block-wide rounds.  The building block is a warp that thins the entries it holds
// in registers to at most 64 that contain its m best: the m-th largest of the 32 lanes' maxima
// (every lane ranks its maximum against the others) is a threshold that at least m entries reach, so everything
// below it can go whichever way ties are broken.  Only when more than 64 entries reach the
// threshold (many equal values, or m close to 32) does the warp take the exact m best instead: the
// m-th largest key by bisection over its bits, ties by bisection over the index bits (a warp-wide
// count per bit).  Values are compared as floats where they are read (maximum, threshold test: two
// or three instructions an entry) and become 32-bit keys whose unsigned order is the selection
// order (key 0 = "no entry") only once they have survived.
//   A  grid (chunks, rows), 8 warps per CTA: each warp loads its share of the CTA's chunk (up to
//      16 or 32 entries per lane) straight into registers and leaves its survivors in shared memory;
//   B  the survivors go to scratch as they are (a second threshold over the whole CTA, from the
//      warps' four largest lane maxima, keeps them to a few dozen), or thinned by warp 0 if more than 64;
//   C  the last CTA of a row to finish (arrival counter) spreads the chunks' survivors over
//      its 8 warps (eight chunks each);  D  its warp 0 thins the warps' survivors once more if more
//      than one warp had any, ranks the at most 64 that remain and writes the first m.
// The row is read from HBM once (4 V bytes).

#include <climits>

#include "common.cuh"

namespace falcon {
namespace {

constexpr int kTopmThreads = 256;
constexpr int kTopmWarps = kTopmThreads / 32;
constexpr int kTopmPerLane = 16;                                  // entries a lane holds in the passes over lists
constexpr int kTopmRowsMax = 32;                                  // entries a lane holds at most in the first pass
constexpr int kTopmChunkMax = kTopmWarps * 32 * kTopmRowsMax;     // 8192 entries per CTA
constexpr int kTopmCap = 64;                                      // entries a thinning pass leaves at most
static_assert(64 * kTopmCap <= kTopmWarps * 32 * kTopmPerLane, "the last CTA's warps hold the survivors of 64 chunks");
static_assert(kTopmWarps * kTopmCap <= 32 * kTopmPerLane, "one warp holds all warps' survivors");
static_assert(FALCON_TOPM_MAX <= 32, "the threshold is the m-th largest of 32 lane maxima");
static_assert(FALCON_TOPM_MAX <= kTopmCap, "the exact selection's m entries fit where the survivors go");

struct TopmParams {
  int32_t n_rows, vocab, m, chunks, chunk_len;
  int32_t warp_span;   // entries of a chunk that one warp takes (a multiple of 32, at most 32 * kTopmRowsMax)
  int32_t cta_thresh;  // pass A also uses a threshold over the whole CTA (see warp_thin_first)
  int64_t logits_stride;
  const float* logits;
  float* top_val;
  int32_t* top_idx;
  uint32_t* part_key;  // [rows, chunks, kTopmCap]
  int32_t* part_idx;   // [rows, chunks, kTopmCap]
  int32_t* part_cnt;   // [rows, chunks] entries in use
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

// The k-th largest (k = 0: the largest) of one value per lane.  Every lane ranks its value against
// all 32 (equal values in lane order, so the ranks are a permutation); the 32 shuffles are
// independent of one another, unlike the stages of a sorting network.
__device__ __forceinline__ uint32_t warp_kth_largest(uint32_t v, int kth, int lane) {
  int rank = 0;
#pragma unroll 4
  for (int j = 0; j < 32; ++j) {
    const uint32_t o = __shfl_sync(0xffffffffu, v, j);
    rank += (o > v || (o == v && j < lane)) ? 1 : 0;
  }
  const unsigned hit = __ballot_sync(0xffffffffu, rank == kth);
  return __shfl_sync(0xffffffffu, v, __ffs(static_cast<int>(hit)) - 1);
}

// Sum of one int per lane over the warp.
__device__ __forceinline__ int warp_sum(int v) { return static_cast<int>(__reduce_add_sync(0xffffffffu, static_cast<unsigned>(v))); }

// The exact cut for the warp's kLen entries per lane (key 0 = none), of which more than m exist:
// t = the m-th largest key, u = the index up to which the entries equal to t belong to the m best.
// An entry is among the m best iff key > t, or key == t and id <= u.
template <int kLen>
__device__ __noinline__ void exact_cut(const uint32_t (&key)[kLen], const int (&id)[kLen], int m, uint32_t& t_out, int& u_out) {
  uint32_t t = 0u;
  for (int bit = 31; bit >= 0; --bit) {
    const uint32_t cand = t | (1u << bit);
    int c = 0;
#pragma unroll
    for (int k = 0; k < kLen; ++k) c += key[k] >= cand ? 1 : 0;
    if (warp_sum(c) >= m) t = cand;
  }
  int above = 0;
#pragma unroll
  for (int k = 0; k < kLen; ++k) above += key[k] > t ? 1 : 0;
  const int need = m - warp_sum(above);  // >= 1 of the entries equal to t
  int u = 0;
  for (int bit = 30; bit >= 0; --bit) {
    const int test = u | ((1 << bit) - 1);  // this bit 0, all lower bits 1
    int c = 0;
#pragma unroll
    for (int k = 0; k < kLen; ++k) c += (key[k] == t && id[k] <= test) ? 1 : 0;
    if (warp_sum(c) < need) u |= 1 << bit;
  }
  t_out = t;
  u_out = u;
}

// Exclusive prefix sum of one count per lane; total = the warp's sum.
__device__ __forceinline__ int warp_offsets(int cnt, int lane, int& total) {
  int incl = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  total = __shfl_sync(0xffffffffu, incl, 31);
  return incl - cnt;
}

// Room for `total` entries in a list shared by the CTA's warps: the position of the first.
__device__ __forceinline__ int warp_reserve(int* fill, int total, int lane) {
  int base = 0;
  if (lane == 0 && total > 0) base = atomicAdd(fill, total);
  return __shfl_sync(0xffffffffu, base, 0);
}

// First pass.  The warp's share of a row's chunk is rowp[0 .. n_w): lane l takes entries l, l + 32,
// ... (kRows at most) as floats, and the survivors (at most kTopmCap) are appended to the list
// out_val / out_id, whose fill count is *fill, as raw values and vocabulary indices (id0 = index
// of rowp[0]).  A NaN is skipped by the maxima and passes the threshold test (it counts as -inf:
// only the later passes, which work on keys, can tell whether it belongs).
template <int kRows>
__device__ __forceinline__ int warp_thin_first(const float* rowp, int n_w, int id0, int m, int lane, float* out_val, int* out_id,
                                               int* fill, uint32_t* cta_top, bool use_cta_top) {
  float x[kRows];
#pragma unroll
  for (int k = 0; k < kRows; ++k) x[k] = (k * 32 + lane < n_w) ? rowp[k * 32 + lane] : -INFINITY;
  // the lane's entries are a prefix of its kRows slots
  const int n_lane = max(0, min(kRows, (n_w - lane + 31) >> 5));
  const uint32_t valid = n_lane >= 32 ? 0xffffffffu : ((1u << n_lane) - 1u);
  float lm = x[0];
#pragma unroll
  for (int k = 1; k < kRows; ++k) lm = fmaxf(lm, x[k]);
  // The warp's threshold and, if asked for, a tighter one for the whole CTA (every warp of the CTA is here
  // then): the four largest lane maxima of each of its 8 warps are 32 different entries, so their m-th
  // largest is reached by at least m entries of the chunk.  With it the CTA's survivors are mostly few enough
  // to go to the row as they are, without a pass of their own: fewer instructions, but a block-wide barrier in
  // the middle of the pass.  The launcher asks for it when the grid is more than one wave (throughput counts);
  // in a single wave the warps are better left to run ahead of one another (60 x 32000: 11.3 against 12.5 us).
  const uint32_t lk = to_key(lm);
  int rank = 0;
#pragma unroll 4
  for (int j = 0; j < 32; ++j) {
    const uint32_t o = __shfl_sync(0xffffffffu, lk, j);
    rank += (o > lk || (o == lk && j < lane)) ? 1 : 0;
  }
  if (rank < 4) cta_top[4 * (threadIdx.x >> 5) + rank] = lk;
  const unsigned hit = __ballot_sync(0xffffffffu, rank == m - 1);
  const uint32_t tau_w = __shfl_sync(0xffffffffu, lk, __ffs(static_cast<int>(hit)) - 1);
  uint32_t tau_c = 0u;
  if (use_cta_top) {
    __syncthreads();
    tau_c = warp_kth_largest(cta_top[lane], m - 1, lane);
  }
  const float tau = from_key(max(tau_w, tau_c));
  uint32_t mask = 0u;
#pragma unroll
  for (int k = 0; k < kRows; ++k)
    if (!(x[k] < tau)) mask |= 1u << k;
  mask &= valid;
  if (warp_sum(__popc(mask)) > kTopmCap) {
    uint32_t key[kRows];
    int id[kRows];
#pragma unroll
    for (int k = 0; k < kRows; ++k) {
      key[k] = ((valid >> k) & 1u) ? to_key(x[k]) : 0u;
      id[k] = id0 + k * 32 + lane;
    }
    uint32_t t;
    int u;
    exact_cut<kRows>(key, id, m, t, u);
    mask = 0u;
#pragma unroll
    for (int k = 0; k < kRows; ++k)
      if (key[k] > t || (key[k] == t && id[k] <= u)) mask |= 1u << k;
  }
  int total;
  int off = warp_offsets(__popc(mask), lane, total) + warp_reserve(fill, total, lane);
  while (mask) {  // one or two entries in most lanes: read them again (L1) instead of indexing registers
    const int k = __ffs(static_cast<int>(mask)) - 1;
    mask &= mask - 1u;
    out_val[off] = rowp[k * 32 + lane];
    out_id[off] = id0 + k * 32 + lane;
    ++off;
  }
  return total;
}

// Later passes: the same on entries that are (key, id) pairs in registers (16 per lane: key 0 =
// none).  The survivors go to out_key / out_id in no particular order: appended to a list shared
// with other warps when `fill` is its fill count, from position 0 when `fill` is null; returns
// their number (the same in every lane).
__device__ __forceinline__ int warp_thin(const uint32_t (&key)[kTopmPerLane], const int (&id)[kTopmPerLane], int m, int lane,
                                         uint32_t* out_key, int* out_id, int* fill) {
  uint32_t lmax = key[0];
#pragma unroll
  for (int k = 1; k < kTopmPerLane; ++k) lmax = max(lmax, key[k]);
  uint32_t tau = warp_kth_largest(lmax, m - 1, lane);
  if (tau == 0u) tau = 1u;  // fewer than m lanes hold anything: keep every entry
  int id_max = INT_MAX;     // entries equal to tau stay if their index is at most this
  int cnt = 0;
#pragma unroll
  for (int k = 0; k < kTopmPerLane; ++k) cnt += key[k] >= tau ? 1 : 0;
  if (warp_sum(cnt) > kTopmCap) {
    exact_cut<kTopmPerLane>(key, id, m, tau, id_max);
    cnt = 0;
#pragma unroll
    for (int k = 0; k < kTopmPerLane; ++k) cnt += (key[k] > tau || (key[k] == tau && id[k] <= id_max)) ? 1 : 0;
  }
  int total;
  int off = warp_offsets(cnt, lane, total) + (fill ? warp_reserve(fill, total, lane) : 0);
#pragma unroll
  for (int k = 0; k < kTopmPerLane; ++k) {
    if (key[k] > tau || (key[k] == tau && id[k] <= id_max)) {
      out_key[off] = key[k];
      out_id[off] = id[k];
      ++off;
    }
  }
  return total;
}

template <int kRows>
__global__ void __launch_bounds__(kTopmThreads, kRows <= 16 ? 4 : 3) tree_topm_kernel(const TopmParams p) {
  // the CTA's list of survivors: pass A appends raw float bits and indices, pass C keys and indices
  __shared__ uint32_t s_key[kTopmWarps * kTopmCap];
  __shared__ int s_id[kTopmWarps * kTopmCap];
  __shared__ uint32_t s_fin_key[kTopmCap];
  __shared__ int s_fin_id[kTopmCap];
  __shared__ uint32_t s_top[4 * kTopmWarps];  // the four largest lane maxima of every warp (pass A)
  __shared__ int s_fill;
  __shared__ int s_last;

  // Under programmatic dependent launch the grid may start while the previous kernel of the stream
  // drains: nothing is read or written before that kernel has completed.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int row = blockIdx.y, chunk = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int c0 = chunk * p.chunk_len;
  const int n = min(p.vocab, c0 + p.chunk_len) - c0;  // >= 1 by construction of the grid
  const float* rowp = p.logits + static_cast<int64_t>(row) * p.logits_stride + c0;
  const int m = p.m;

  if (tid == 0) s_fill = 0;
  __syncthreads();

  // ---- A: each warp thins its share of the chunk (coalesced 128-byte loads, all in flight at once) ----
  {
    const int w0 = warp * p.warp_span;
    const int n_w = max(0, min(p.warp_span, n - w0));
    warp_thin_first<kRows>(rowp + w0, n_w, c0 + w0, m, lane, reinterpret_cast<float*>(s_key), s_id, &s_fill, s_top, p.cta_thresh != 0);
  }
  __syncthreads();

  // The CTA's list, 16 entries per lane of one warp (raw: it holds raw values, which become keys here).
  auto from_list = [&](uint32_t (&key)[kTopmPerLane], int (&id)[kTopmPerLane], bool raw) {
    const int fill = s_fill;
#pragma unroll
    for (int k = 0; k < kTopmPerLane; ++k) {
      const int j = k * 32 + lane;
      const bool in = j < fill;
      const uint32_t v = in ? s_key[j] : 0u;
      key[k] = in ? (raw ? to_key(__uint_as_float(v)) : v) : 0u;
      id[k] = in ? s_id[j] : 0;
    }
  };

  // ---- B: the CTA's survivors go to the row: as they are when they are few enough, else thinned by warp 0 ----
  const int64_t po = static_cast<int64_t>(row) * p.chunks + chunk;
  const int fill_a = s_fill;
  if (fill_a <= kTopmCap) {
    if (tid < fill_a) {
      p.part_key[po * kTopmCap + tid] = to_key(__uint_as_float(s_key[tid]));
      p.part_idx[po * kTopmCap + tid] = s_id[tid];
    }
    __syncthreads();  // every thread's entries before thread 0's fence
    if (tid == 0) {
      p.part_cnt[po] = fill_a;
      s_fill = 0;
      __threadfence();
      s_last = (atomicAdd(&p.tickets[row], 1) == p.chunks - 1);
    }
  } else if (warp == 0) {
    uint32_t key[kTopmPerLane];
    int id[kTopmPerLane];
    from_list(key, id, true);
    const int cnt = warp_thin(key, id, m, lane, p.part_key + po * kTopmCap, p.part_idx + po * kTopmCap, nullptr);
    __syncwarp();  // every lane's entries before lane 0's fence
    if (lane == 0) {
      p.part_cnt[po] = cnt;
      s_fill = 0;  // (the list is in registers: pass C may refill it)
      __threadfence();
      s_last = (atomicAdd(&p.tickets[row], 1) == p.chunks - 1);
    }
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();

  // ---- C: last CTA of the row: the chunks' survivors, eight chunks per warp ----
  {
    const int64_t ro = static_cast<int64_t>(row) * p.chunks;
    uint32_t key[kTopmPerLane];
    int id[kTopmPerLane];
    int cn[kTopmPerLane / 2];
#pragma unroll
    for (int c = 0; c < kTopmPerLane / 2; ++c) {
      const int ch = warp * (kTopmPerLane / 2) + c;
      cn[c] = ch < p.chunks ? __ldcg(p.part_cnt + ro + ch) : 0;
    }
#pragma unroll
    for (int k = 0; k < kTopmPerLane; ++k) {
      // entry k * 32 + lane of this warp: chunk k / 2 of its eight, slot (k & 1) * 32 + lane
      const int slot = (k & 1) * 32 + lane;
      const bool in = slot < cn[k >> 1];
      const int64_t at = (ro + warp * (kTopmPerLane / 2) + (k >> 1)) * kTopmCap + slot;
      key[k] = in ? __ldcg(p.part_key + at) : 0u;
      id[k] = in ? __ldcg(p.part_idx + at) : 0;
    }
    if (warp * (kTopmPerLane / 2) < p.chunks) warp_thin(key, id, m, lane, s_key, s_id, &s_fill);
  }
  __syncthreads();

  // ---- D: warp 0 thins once more (when several warps had chunks), ranks what is left and writes
  // the row's result ----
  if (warp == 0) {
    const uint32_t* fin_key = s_key;
    const int* fin_id = s_id;
    int cnt = s_fill;
    if (p.chunks > kTopmPerLane / 2) {
      uint32_t key[kTopmPerLane];
      int id[kTopmPerLane];
      from_list(key, id, false);
      cnt = warp_thin(key, id, m, lane, s_fin_key, s_fin_id, nullptr);
      fin_key = s_fin_key;
      fin_id = s_fin_id;
    }
    __syncwarp();
    // At most 64 entries, two per lane: an entry's place in the result is the number of entries that
    // come before it (the entries are distinct, so the places are too).
    const uint64_t e0 = lane < cnt ? entry(fin_key[lane], fin_id[lane]) : 0ull;
    const uint64_t e1 = lane + 32 < cnt ? entry(fin_key[lane + 32], fin_id[lane + 32]) : 0ull;
    int r0 = 0, r1 = 0;
    for (int j = 0; j < cnt; ++j) {
      const uint64_t o = entry(fin_key[j], fin_id[j]);
      r0 += o > e0 ? 1 : 0;
      r1 += o > e1 ? 1 : 0;
    }
    if (e0 != 0ull && r0 < m) {
      p.top_val[static_cast<int64_t>(row) * m + r0] = from_key(static_cast<uint32_t>(e0 >> 32));
      p.top_idx[static_cast<int64_t>(row) * m + r0] = static_cast<int>(~static_cast<uint32_t>(e0));
    }
    if (e1 != 0ull && r1 < m) {
      p.top_val[static_cast<int64_t>(row) * m + r1] = from_key(static_cast<uint32_t>(e1 >> 32));
      p.top_idx[static_cast<int64_t>(row) * m + r1] = static_cast<int>(~static_cast<uint32_t>(e1));
    }
    if (lane == 0) p.tickets[row] = 0;  // ready for the next call
  }
}

}  // namespace

int launch_tree_topm(falcon_ctx* ctx, const falcon_topm_args& a, cudaStream_t s) {
  const int N = a.n_rows;
  if (N > 65535) return FALCON_ERR_CAPACITY;
  // As many CTAs as are resident at once (four per SM) where the vocabulary allows; a chunk is at
  // most what a CTA holds in registers, split evenly over its warps in units of 32 entries.
  int chunks = 4 * ctx->sm_count / N;
  if (chunks < 1) chunks = 1;
  const int max_chunks = (a.vocab + 2047) / 2048;
  if (chunks > max_chunks) chunks = max_chunks;
  if (chunks > kTopmPerLane / 2) chunks = kTopmPerLane / 2;  // one warp of the row's last CTA then holds all survivors
  const int min_chunks = (a.vocab + kTopmChunkMax - 1) / kTopmChunkMax;
  if (chunks < min_chunks) chunks = min_chunks;
  if (chunks > 64) return FALCON_ERR_CAPACITY;  // vocabulary beyond 64 x 8192 entries
  int chunk_len = (a.vocab + chunks - 1) / chunks;
  int warp_span = ((chunk_len + kTopmWarps - 1) / kTopmWarps + 31) & ~31;
  if (warp_span > 32 * kTopmRowsMax) warp_span = 32 * kTopmRowsMax;
  chunk_len = kTopmWarps * warp_span;  // (the last chunk of a row may be shorter or, rounded up, missing)
  chunks = (a.vocab + chunk_len - 1) / chunk_len;

  const size_t part = static_cast<size_t>(N) * chunks * kTopmCap;
  int rc = ensure_workspace(ctx, part * 8 + static_cast<size_t>(N) * chunks * 4 + 256);
  if (rc) return rc;
  rc = ensure_tickets(ctx, N, s);
  if (rc) return rc;

  TopmParams p;
  p.n_rows = N;
  p.vocab = a.vocab;
  p.m = a.m;
  p.chunks = chunks;
  p.chunk_len = chunk_len;
  p.warp_span = warp_span;
  // (CTAs resident per SM: 4 with 16 entries per lane, 3 with 32: the kernel's launch bounds)
  p.cta_thresh = static_cast<int64_t>(N) * chunks > static_cast<int64_t>(warp_span <= 16 * 32 ? 4 : 3) * ctx->sm_count ? 1 : 0;
  p.logits_stride = a.logits_stride;
  p.logits = a.logits;
  p.top_val = a.top_val;
  p.top_idx = a.top_idx;
  p.part_key = static_cast<uint32_t*>(ctx->ws);
  p.part_idx = reinterpret_cast<int32_t*>(static_cast<uint32_t*>(ctx->ws) + part);
  p.part_cnt = p.part_idx + part;
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
  cudaError_t e = warp_span <= 16 * 32 ? cudaLaunchKernelEx(&cfg, tree_topm_kernel<16>, p)
                                       : cudaLaunchKernelEx(&cfg, tree_topm_kernel<kTopmRowsMax>, p);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "tree_topm_kernel launch");
  return FALCON_OK;
}

}  // namespace falcon
