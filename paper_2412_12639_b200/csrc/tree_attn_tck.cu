// falcon_tree_attn, tensor-core kernel with the KEYS on the tensor-memory lanes (head_dim 128, tree
// K/V in the cache).
//
// A verification tree has few query rows (60-80 nodes x the query heads of one KV head) and many
// keys, so the score tile is computed transposed: S^T = K_tile . Q^T with the 128 keys of a tile on
// the M side (one key per TMEM lane) and the query rows on the N side, which tcgen05.mma sizes in
// steps of 16 (60 nodes -> N = 64, 80 -> 80), and O^T += V_tile^T . P^T.  Every lane of every
// softmax warp then holds a real key, a query row's accumulator is one TMEM column whatever key
// contributed to it, and the warps of a lane quadrant share a tile by taking different query
// columns, with no state in common.
//
// Work decomposition: one thread-block cluster per (sequence, KV head, block of query rows); row r
// of a KV head is (tree node r / G, query head r % G).  The cluster's CTAs split the key range
// (prefix + tree) into runs of whole 128-key tiles, and their partial results are summed through
// distributed shared memory (each CTA owns a share of the rows).
//
// Softmax without a running maximum: every CTA subtracts the same per-row reference, the row's
// score against cache row 0, which all CTAs can compute before their first tile arrives.  fp32
// carries exponents up to 2^127, so a weight p = 2^(score - reference) needs no rescaling as long as
// the row's scores stay within about 2^100 of the reference; then the partial results of the
// splits add up without weights.  A row whose normaliser leaves [2^-100, 2^100] (or is not finite)
// is recomputed from global memory by one warp with an exact running maximum (rare: it takes
// scores hundreds of units apart).
//
// Inside a CTA (576 threads):
//   warp 0     TMA producer: Q block, then K and V tiles (128 keys, 128-byte swizzle) into a ring.
//   warp 1     one elected lane issues tcgen05.mma: S^T(j) = K(j).Q^T into one of two TMEM score
//              buffers, O^T += V(j)^T.P(j)^T with P^T read from shared memory.
//   warps 2-17 softmax: warp w works on TMEM lane quadrant w % 4 (32 keys) and on the 16-column
//              chunks (w - 2) / 4, + 4, ... of the query rows: tcgen05.ld, p = 2^(s.scale - ref),
//              tree mask from the key's descendant bit set, row sums in registers, P^T as bf16 into
//              the shared memory of the K tile it was computed from (free once S^T exists).
// All three falcon kernels are launched programmatically dependent; set-up that touches no global
// memory, and prefix tiles the caller declared stable, come before griddepcontrol.wait.
// Every mbarrier wait is bounded; a wait that runs out sets FALCON_DEV_TIMEOUT.
#include "tc_util.cuh"

// Profiling hooks, empty by default: a private build may predefine them to record time stamps.
#ifndef FALCON_TRACE
#define FALCON_TRACE(who, id)
#define FALCON_TRACE_PARAMS
#define FALCON_TRACE_LAUNCH(p)
#endif

namespace falcon {
namespace {
using namespace tc;

constexpr int kD = 128;
constexpr int kBK = 128;                        // keys per tile = TMEM lanes
constexpr int kCW = 16;                         // query columns per softmax chunk
constexpr int kColGroups = 4;                   // softmax warps per lane quadrant
constexpr int kSmWarps = 4 * kColGroups;
constexpr int kSmThreads = 32 * kSmWarps;       // 512
constexpr int kThreads = 32 * (2 + kSmWarps);   // 576
constexpr int kWarpProducer = 0;
constexpr int kWarpMma = 1;
constexpr int kWarpSm0 = 2;
constexpr int kMaxSplits = 8;
constexpr int kHostSeqs = 8;
constexpr uint32_t kTileBytes = kBK * kD * 2;   // 32 KB: two 64-column halves of 16 KB
constexpr uint32_t kHalfTile = kBK * 128;       // 16 KB
constexpr uint32_t kStageBytes = 2 * kTileBytes;
constexpr int kPartRows = kD + 2;               // a CTA's partial result: 128 head-dim rows, 2 rows for the row sums
constexpr float kLMin = 7.8886090522101181e-31f;  // 2^-100
constexpr float kLMax = 1.2676506002282294e+30f;  // 2^100
constexpr uint32_t kMrgSpin = 1u << 26;         // tries of the one wait that must not give up early
#ifndef FALCON_TCK_EARLY
#define FALCON_TCK_EARLY 3
#endif
constexpr int kEarlyTiles = FALCON_TCK_EARLY;   // prefix tiles requested before the grid dependency wait, at most

enum {
  kBarQ = 0,
  kBarKVFull = 1,                    // [3]
  kBarKVEmpty = kBarKVFull + 3,      // [3]
  kBarSFull = kBarKVEmpty + 3,       // [2]
  kBarPFull = kBarSFull + 2,         // [2]
  kBarODone = kBarPFull + 2,
  kBarMrg = kBarODone + 1,
  kNumBars = kBarMrg + 1
};

// kChunks = 1: up to 64 query rows per unit (3-stage ring, 256 TMEM columns);
// kChunks = 2: up to 128 (2-stage ring, 512 columns).
template <int kChunks>
struct Cfg {
  static constexpr int kN = 64 * kChunks;
  static constexpr int kStages = kChunks == 1 ? 3 : 2;
  static constexpr uint32_t kTmemCols = 256 * kChunks;
  static constexpr uint32_t kColStride = 64 * kChunks;   // S^T(0), S^T(1), O^T, row sums
  static constexpr uint32_t kQBytes = kN * kD * 2;
  static constexpr uint32_t kOffQ = 0;
  static constexpr uint32_t kOffKV = kOffQ + kQBytes;
  static constexpr uint32_t kOffMrg = kOffKV + kStages * kStageBytes;
  // What a CTA can receive: from each of the other splits its share of the head-dim rows plus the two
  // row-sum rows.  The launcher keeps (splits - 1) * (ceil(128 / splits) + 2) * pitch within this.
  static constexpr uint32_t kMrgBytes = kChunks == 1 ? 17408 : 40960;
  static constexpr uint32_t kOffDesc = kOffMrg + kMrgBytes;               // [128 tree keys][kN / 32] words
  static constexpr uint32_t kDescWords = kN / 32;
  static constexpr uint32_t kOffRef = kOffDesc + 128 * kDescWords * 4;   // [kN] fp32: reference, later 1 / row sum
  static constexpr uint32_t kOffRescue = kOffRef + kN * 4;               // [kN] bytes
  static constexpr uint32_t kOffPar = kOffRescue + kN;                   // [128] int8: the tree's parent array
  static constexpr uint32_t kOffOnes = kOffPar + 128;                    // 256 bytes of bf16 1.0 (see kernel)
  static constexpr uint32_t kOffBars = kOffOnes + 256;
  static constexpr uint32_t kOffMisc = kOffBars + 8 * kNumBars;          // tmem base, abort flag
  static constexpr uint32_t kSmemBytes = kOffMisc + 16;
  // used once the main loop is over
  static constexpr uint32_t kOffStage = 0;                                // [kPartRows][pitch] this CTA's partial result
  static_assert(kPartRows * (kN * 2 + 16) <= kOffMrg, "staging lies over Q and the ring");
  static_assert(kSmemBytes <= 232448, "shared memory per CTA");
};

// bytes between the rows of a partial result of n query columns: an odd number of 16-byte units, so
// that 16-byte accesses of consecutive rows fall into different banks
__host__ __device__ constexpr uint32_t part_pitch(int n) { return static_cast<uint32_t>(n) * 2u + 16u; }

struct TckParams {
  int32_t Hq, Hkv, G, g_shift, s_cap, total_nodes;
  int32_t n_rows;          // query rows per unit (multiple of 16, at most Cfg::kN)
  uint32_t idesc_qk, idesc_pv, idesc_sum;
  float scale_log2;
  const int32_t* node_off;
  const int32_t* parent;
  const int32_t* prefix_len;
  int32_t* status;
  const uint64_t* tree_mask;
  const __nv_bfloat16* q;
  const __nv_bfloat16* k;
  const __nv_bfloat16* v;
  int64_t kv_stride_b, kv_stride_h, kv_stride_s;
  __nv_bfloat16* out;
  int32_t have_host;
  int32_t early_prefix;
  int32_t h_node_off[kHostSeqs + 1];
  int32_t h_prefix[kHostSeqs];
  FALCON_TRACE_PARAMS
};

// Shared-memory matrix descriptor without swizzle: 8 x 16-byte core matrices, `lbo` bytes between
// the two core matrices of a K step, `sbo` bytes between 8-row groups.
__device__ __forceinline__ uint64_t smem_desc_plain(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return static_cast<uint64_t>((addr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(lbo_bytes >> 4) << 16) |
         (static_cast<uint64_t>(sbo_bytes >> 4) << 32) | (1ull << 46);
}

// 16 bytes into the shared memory of a CTA of the cluster (this one included); the store counts 16
// bytes on the mbarrier `bar`, which must live in the same CTA as the destination.
__device__ __forceinline__ void st_async_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(addr),
               "r"(a), "r"(b), "r"(c), "r"(d), "r"(bar)
               : "memory");
}
// Bounded wait with cluster-scope acquire, for a whole warp.
__device__ __forceinline__ bool mbar_wait_cluster_warp(uint32_t bar, uint32_t parity) {
  bool done = false;
  for (uint32_t it = 0; it < kMrgSpin && !done; ++it) {
    uint32_t ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    done = __all_sync(0xffffffffu, ok != 0);
  }
  return done;
}

__device__ __forceinline__ float bf16lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf16hi(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }

// One query row recomputed exactly by a warp from global memory (running maximum in fp32): the
// fallback for rows whose scores lie too far from the reference for the fast path.
__device__ void rescue_row(const TckParams& p, int b, int kvh, int node_base, int T, int Lc, int S_valid, int mg,
                           int lane) {
  const int node = mg >> p.g_shift, head = kvh * p.G + (mg & (p.G - 1));
  uint64_t lo = 0, hi = 0;
  if (p.tree_mask) {
    lo = p.tree_mask[2 * static_cast<int64_t>(node_base + node)];
    hi = p.tree_mask[2 * static_cast<int64_t>(node_base + node) + 1];
  } else {
    ancestor_mask(p.parent + node_base, T, node, lo, hi);
  }
  const uint2 qv = *reinterpret_cast<const uint2*>(p.q + (static_cast<int64_t>(node_base + node) * p.Hq + head) * kD + 4 * lane);
  const float q0 = bf16lo(qv.x), q1 = bf16hi(qv.x), q2 = bf16lo(qv.y), q3 = bf16hi(qv.y);
  const __nv_bfloat16* kb = p.k + b * p.kv_stride_b + kvh * p.kv_stride_h + 4 * lane;
  const __nv_bfloat16* vb = p.v + b * p.kv_stride_b + kvh * p.kv_stride_h + 4 * lane;
  float m = -INFINITY, l = 0.f, a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
  for (int key = 0; key < S_valid; ++key) {
    if (key >= Lc && !bit128(lo, hi, key - Lc)) continue;
    const uint2 kk = *reinterpret_cast<const uint2*>(kb + key * p.kv_stride_s);
    float s = q0 * bf16lo(kk.x);
    s = fmaf(q1, bf16hi(kk.x), s);
    s = fmaf(q2, bf16lo(kk.y), s);
    s = fmaf(q3, bf16hi(kk.y), s);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    s *= p.scale_log2;
    const float mn = fmaxf(m, s);
    const float alpha = ex2(m - mn), pw = ex2(s - mn);
    const uint2 vv = *reinterpret_cast<const uint2*>(vb + key * p.kv_stride_s);
    l = fmaf(l, alpha, pw);
    a0 = fmaf(a0, alpha, pw * bf16lo(vv.x));
    a1 = fmaf(a1, alpha, pw * bf16hi(vv.x));
    a2 = fmaf(a2, alpha, pw * bf16lo(vv.y));
    a3 = fmaf(a3, alpha, pw * bf16hi(vv.y));
    m = mn;
  }
  const float inv = l > 0.f ? 1.f / l : 0.f;
  const __nv_bfloat162 h0 = __floats2bfloat162_rn(a0 * inv, a1 * inv), h1 = __floats2bfloat162_rn(a2 * inv, a3 * inv);
  uint2 o;
  o.x = *reinterpret_cast<const uint32_t*>(&h0);
  o.y = *reinterpret_cast<const uint32_t*>(&h1);
  *reinterpret_cast<uint2*>(p.out + (static_cast<int64_t>(node_base + node) * p.Hq + head) * kD + 4 * lane) = o;
}

template <int kChunks>
__global__ void __launch_bounds__(kThreads, 1)
tree_attn_tck_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                     const TckParams p) {
  using C = Cfg<kChunks>;
  constexpr int kStages = C::kStages;
  extern __shared__ __align__(1024) unsigned char smem_gen[];
  const uint32_t smem_base = smem_u32(smem_gen);
  uint32_t* s_desc = reinterpret_cast<uint32_t*>(smem_gen + C::kOffDesc);
  float* s_ref = reinterpret_cast<float*>(smem_gen + C::kOffRef);
  unsigned char* s_rescue = smem_gen + C::kOffRescue;
  signed char* s_par = reinterpret_cast<signed char*>(smem_gen + C::kOffPar);
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(smem_gen + C::kOffMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + C::kOffMisc + 4);
  const uint32_t bars = smem_base + C::kOffBars;
  auto bar = [&](int i) { return bars + 8u * static_cast<uint32_t>(i); };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_splits = gridDim.x, split = blockIdx.x;  // cluster = all CTAs of a row of the grid
  const int kvh = blockIdx.y % p.Hkv, mtile = blockIdx.y / p.Hkv, b = blockIdx.z;
  const int G = p.G, N = p.n_rows, n_chunks = N >> 4;
  const uint32_t q_half_bytes = static_cast<uint32_t>(N) * 128u;  // between the two 64-column halves of Q
  FALCON_TRACE(tid == 0, 0);
  {
    // The kernel's parameters live in constant memory that is rewritten for every launch, so the
    // first access to each of its 64-byte lines is a round trip to L2.  Touch every line now, where
    // the latency overlaps the previous kernel, instead of where its values are needed.
    const uint32_t warm = static_cast<uint32_t>(p.Hq) ^ static_cast<uint32_t>(reinterpret_cast<uintptr_t>(p.tree_mask)) ^
                          static_cast<uint32_t>(reinterpret_cast<uintptr_t>(p.q)) ^ static_cast<uint32_t>(p.kv_stride_s) ^
                          static_cast<uint32_t>(reinterpret_cast<uintptr_t>(p.out)) ^ static_cast<uint32_t>(p.h_node_off[2]) ^
                          static_cast<uint32_t>(p.h_prefix[kHostSeqs - 1]);
    asm volatile("" ::"r"(warm));
  }

  // ---- set-up that touches no global memory (overlaps the previous kernel under programmatic launch) ----
  if (warp == kWarpProducer) {
    if (lane == 0) {
      *abort_flag = (smem_base & 1023u) ? 1 : 0;  // the swizzled tiles need a 1 KB aligned base
      prefetch_tmap(&tm_k);
      prefetch_tmap(&tm_v);
    }
    if (lane < kNumBars)
      mbar_init(bar(lane), (lane == kBarPFull || lane == kBarPFull + 1 || lane == kBarQ) ? kSmWarps : 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncwarp();
  } else if (warp == kWarpMma) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem_base)),
                 "r"(C::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  } else {
    const int st_id = tid - 32 * kWarpSm0;
    for (int i = st_id; i < 128 * static_cast<int>(C::kDescWords); i += kSmThreads) s_desc[i] = 0u;
    if (st_id < C::kN) s_rescue[st_id] = 0;
    if (st_id < 64) reinterpret_cast<uint32_t*>(smem_gen + C::kOffOnes)[st_id] = 0x3f803f80u;  // bf16 1.0 pairs
    fence_async_smem();
  }

  // Geometry of this CTA's share, from the sequence's node range and prefix length.
  int node_base = 0, T_real = 0, L_raw = 0;
  int T, rows_total, n_valid, L, Lc, S_valid, tile_begin, tile_end, n_my, key_begin;
  auto geometry = [&]() {
    T = min(T_real, FALCON_T_MAX);
    rows_total = T * G;
    n_valid = min(N, rows_total - mtile * N);
    L = max(L_raw, 0);
    Lc = min(L, p.s_cap);
    S_valid = min(L + T, p.s_cap);  // keys that exist below the cache capacity
    // Whole tiles per split, boundaries rounded up: a longer run goes to an early split, the last
    // one has the tree's tiles, whose masked pass is the slowest.
    const int n_tiles = (S_valid + kBK - 1) / kBK;
    tile_begin = (split * n_tiles + n_splits - 1) / n_splits;
    tile_end = ((split + 1) * n_tiles + n_splits - 1) / n_splits;
    n_my = tile_end - tile_begin;
    key_begin = tile_begin * kBK;
  };
  auto load_tile = [&](int j) {
    const int st = j % kStages;
    const uint32_t dst = smem_base + C::kOffKV + st * kStageBytes;
    mbar_expect_tx(bar(kBarKVFull + st), kStageBytes);
    tma_load_5d(dst, &tm_k, bar(kBarKVFull + st), 0, key_begin + j * kBK, 0, kvh, b);
    tma_load_5d(dst + kTileBytes, &tm_v, bar(kBarKVFull + st), 0, key_begin + j * kBK, 0, kvh, b);
  };
  // This thread's piece of the Q block (softmax threads): 16 head-dim columns of one or two rows.
  const int st_id = tid - 32 * kWarpSm0;
  const int q_part = st_id & 7;
  auto q_piece = [&](int r) -> const __nv_bfloat16* {
    const int mg = mtile * N + r;
    return p.q + (static_cast<int64_t>(node_base + (mg >> p.g_shift)) * p.Hq + kvh * G + (mg & (G - 1))) * kD + q_part * 16;
  };
  int n_early = 0;  // K/V tiles requested before the wait below
  if (p.have_host) {
    node_base = p.h_node_off[b];
    T_real = p.h_node_off[b + 1] - node_base;
    L_raw = p.h_prefix[b];
    geometry();
    if (n_valid > 0) {
      if (warp == kWarpProducer && lane == 0 && p.early_prefix) {
        // Prefix rows that the caller declares stable (written before the kernel that precedes this
        // one in the stream started) may be requested while that kernel is still finishing.
        for (int j = 0; j < min(n_my, min(kStages, kEarlyTiles)) && key_begin + (j + 1) * kBK <= Lc; ++j) {
          load_tile(j);
          ++n_early;
        }
      }
      if (warp >= kWarpSm0 && n_my > 0) {
        // hints only (q and a tree's first row may still be being written): have the Q block and the
        // reference key on their way into L2
#pragma unroll
        for (int pass = 0; pass < kChunks; ++pass) {
          const int r = (st_id >> 3) + 64 * pass;
          if (r < n_valid) asm volatile("prefetch.global.L2 [%0];" ::"l"(q_piece(r)));
        }
        if (st_id < 8) asm volatile("prefetch.global.L2 [%0];" ::"l"(p.k + b * p.kv_stride_b + kvh * p.kv_stride_h + st_id * 16));
        // and the address translation of the output rows this CTA will write
        if (st_id >= 64 && st_id - 64 < n_valid) {
          const int mg = mtile * N + st_id - 64;
          asm volatile("prefetch.global.L2 [%0];" ::"l"(
              p.out + (static_cast<int64_t>(node_base + (mg >> p.g_shift)) * p.Hq + kvh * G + (mg & (G - 1))) * kD));
        }
      }
    }
  }
  // Everything below may read what earlier kernels of the stream wrote and writes `out`.
  FALCON_TRACE(tid == 0, 1);
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  FALCON_TRACE(tid == 0, 2);
  if (!p.have_host) {
    node_base = p.node_off[b];
    T_real = p.node_off[b + 1] - node_base;
    L_raw = p.prefix_len[b];
    geometry();
  }
  if (n_valid <= 0) {  // no query rows here; same decision in every CTA of the cluster
    tc_fence_before();
    __syncthreads();
    if (warp == kWarpMma) {
      tc_fence_after();
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(*s_tmem_base), "r"(C::kTmemCols)
                   : "memory");
    }
    return;
  }
  // The softmax threads' global loads go out first: Q (plain loads: a TMA request would queue behind
  // the K/V tiles already asked for), the reference key (cache row 0) and the tree's parent array.
  uint4 qreg[kChunks][2], kref[2];
  int par_raw = -1;
  const bool has_tree_keys = tile_end * kBK > Lc;
  const bool need_tree = has_tree_keys || (split == 0 && kvh == 0);  // the latter reports malformed trees
  if (warp >= kWarpSm0 && n_my > 0) {
#pragma unroll
    for (int pass = 0; pass < kChunks; ++pass) {
      const int r = (st_id >> 3) + 64 * pass;
      qreg[pass][0] = qreg[pass][1] = make_uint4(0u, 0u, 0u, 0u);
      if (r < n_valid) {
        qreg[pass][0] = reinterpret_cast<const uint4*>(q_piece(r))[0];
        qreg[pass][1] = reinterpret_cast<const uint4*>(q_piece(r))[1];
      }
    }
    const __nv_bfloat16* k0p = p.k + b * p.kv_stride_b + kvh * p.kv_stride_h + q_part * 16;
    kref[0] = reinterpret_cast<const uint4*>(k0p)[0];
    kref[1] = reinterpret_cast<const uint4*>(k0p)[1];
    if (need_tree && !p.tree_mask && st_id < T) par_raw = p.parent[node_base + st_id];
  }

  // merge geometry: CTA `rank` owns head-dim rows [rank * d_per, ...) of the unit's result
  const uint32_t pitch = part_pitch(N);
  const int d_per = (kD + n_splits - 1) / n_splits;
  const int d0 = split * d_per;
  const int d_mine = max(0, min(kD, d0 + d_per) - d0);
  const uint32_t slot_bytes = static_cast<uint32_t>(d_per + 2) * pitch;

  if (warp == kWarpProducer && lane == 0) {
    // every split (this one included) delivers its share of this CTA's head-dim rows and the row sums
    mbar_expect_tx(bar(kBarMrg), static_cast<uint32_t>(n_splits * (d_mine + 2) * N * 2));
    for (int j = n_early; j < min(n_my, kStages); ++j) load_tile(j);
    if (split == 0 && mtile == 0 && kvh == 0 && (L + T > p.s_cap || T_real > FALCON_T_MAX))
      dev_status_or(p.status, b, FALCON_DEV_CAPACITY);
    FALCON_TRACE(true, 3);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  FALCON_TRACE(tid == 0, 4);
  const uint32_t tmem_base = *s_tmem_base;
  // Cluster phase 1: "my merge barrier exists".  Arrive now, wait just before the first remote copy.
  if (n_splits > 1) cluster_arrive();

  if (warp == kWarpProducer) {
    // ================================ TMA producer (ring refills) ================================
    if (lane == 0) {
      for (int j = kStages; j < n_my; ++j) {
        if (!mbar_wait(bar(kBarKVEmpty + j % kStages), (j / kStages - 1) & 1, abort_flag)) break;
        load_tile(j);
      }
    }
  } else if (warp == kWarpMma) {
    // ================================ MMA issuer ================================
    if (n_my > 0) {
      uint32_t elected;
      asm volatile("{ .reg .pred p; elect.sync _|p, 0xffffffff; selp.u32 %0, 1, 0, p; }" : "=r"(elected));
      bool ok = mbar_wait_warp(bar(kBarQ), 0, abort_flag);
      FALCON_TRACE(elected, 5);
      auto issue_qk = [&](int j) -> bool {
        const int st = j % kStages, sb = j & 1;
        if (!mbar_wait_warp(bar(kBarKVFull + st), (j / kStages) & 1, abort_flag)) return false;
        FALCON_TRACE(elected && j < 4, 10 + 4 * j);
        tc_fence_after();
        const uint32_t kbase = smem_base + C::kOffKV + st * kStageBytes;
        if (elected) {
#pragma unroll
          for (int kk = 0; kk < kD / 16; ++kk) {
            // K tile (A) and Q block (B): K-major, 16 head-dim columns = 32 bytes inside the 128-byte swizzle row
            const uint64_t ad = smem_desc(kbase + (kk >> 2) * kHalfTile + (kk & 3) * 32, 16, 1024);
            const uint64_t bd = smem_desc(smem_base + C::kOffQ + (kk >> 2) * q_half_bytes + (kk & 3) * 32, 16, 1024);
            umma_bf16_ss(tmem_base + sb * C::kColStride, ad, bd, p.idesc_qk, kk > 0 ? 1u : 0u);
          }
          umma_commit(bar(kBarSFull + sb));
        }
        __syncwarp();
        return true;
      };
      auto issue_pv = [&](int t) {
        const int st = t % kStages;
        const uint32_t pbase = smem_base + C::kOffKV + st * kStageBytes;   // P^T lies over the K tile
        const uint32_t vbase = pbase + kTileBytes;
        // keys of the tile that exist, in MMA steps of 16 (rows above them hold zeros in P^T and V)
        const int nk = (min(kBK, S_valid - (key_begin + t * kBK)) + 15) >> 4;
        if (elected) {
          for (int kk = 0; kk < nk; ++kk) {
            // V^T (A) and P^T (B): both with the M / N index contiguous; 16 keys = 2 KB, the 64-column
            // blocks of either operand 16 KB apart
            const uint64_t ad = smem_desc(vbase + kk * 2048, kHalfTile, 1024);
            const uint64_t bd = smem_desc(pbase + kk * 2048, kHalfTile, 1024);
            umma_bf16_ss(tmem_base + 2 * C::kColStride, ad, bd, p.idesc_pv, (t > 0 || kk > 0) ? 1u : 0u);
          }
          // Row sums on the tensor core as well: an all-ones A (every row and both K halves read the
          // same 16-byte rows of ones, strides zero and 128) times P^T gives, in every TMEM lane, the
          // sum over the tile's keys of exactly the bf16 weights the accumulator received.
          const uint64_t od = smem_desc_plain(smem_base + C::kOffOnes, 128, 0);
          for (int kk = 0; kk < nk; ++kk) {
            const uint64_t bd = smem_desc(pbase + kk * 2048, kHalfTile, 1024);
            umma_bf16_ss(tmem_base + 3 * C::kColStride, od, bd, p.idesc_sum, (t > 0 || kk > 0) ? 1u : 0u);
          }
          umma_commit(bar(kBarKVEmpty + st));
        }
        __syncwarp();
      };
      // Two tiles of scores are always in flight.  When P^T(t) is there, score buffer t & 1 has been
      // read, so the scores of tile t+2 can go into it.
      ok = ok && issue_qk(0);
      if (ok && n_my > 1) ok = issue_qk(1);
      for (int t = 0; ok && t < n_my; ++t) {
        if (!mbar_wait_warp(bar(kBarPFull + (t & 1)), (t >> 1) & 1, abort_flag)) { ok = false; break; }
        FALCON_TRACE(elected && t < 4, 11 + 4 * t);
        tc_fence_after();
        issue_pv(t);
        if (t + 2 < n_my) ok = issue_qk(t + 2);
      }
      if (elected) umma_commit(bar(kBarODone));  // fires once every MMA issued so far has finished
      __syncwarp();
    }
  } else {
    // ================================ softmax warps ================================
    const int q4 = warp & 3;                       // TMEM lane quadrant this warp can reach
    const int grp = (warp - kWarpSm0) >> 2;        // first 16-column chunk of this warp
    const int kr = q4 * 32 + lane;                 // key row inside a tile; head-dim row of O^T in the epilogue
    const uint32_t tmem_lane = tmem_base + (static_cast<uint32_t>(q4 * 32) << 16);
    bool live = n_my > 0 && !*abort_flag;

    if (live) {
      // (a) Q block into shared memory in the layout the MMA reads (K-major rows of 128 bytes per
      // 64-column half, 16-byte units XOR-swizzled by the row), and the reference of every query
      // row: its scaled score against cache row 0 (8 threads per row, 16 columns each).
      const uint32_t kw[8] = {kref[0].x, kref[0].y, kref[0].z, kref[0].w, kref[1].x, kref[1].y, kref[1].z, kref[1].w};
#pragma unroll
      for (int pass = 0; pass < kChunks; ++pass) {
        const int r = (st_id >> 3) + 64 * pass;
        if (r < N) {
          unsigned char* qrow = smem_gen + C::kOffQ + (q_part >> 2) * q_half_bytes + r * 128;
          const int u0 = 2 * (q_part & 3);
          *reinterpret_cast<uint4*>(qrow + ((u0 ^ (r & 7)) << 4)) = qreg[pass][0];
          *reinterpret_cast<uint4*>(qrow + (((u0 + 1) ^ (r & 7)) << 4)) = qreg[pass][1];
          const uint32_t qw[8] = {qreg[pass][0].x, qreg[pass][0].y, qreg[pass][0].z, qreg[pass][0].w,
                                  qreg[pass][1].x, qreg[pass][1].y, qreg[pass][1].z, qreg[pass][1].w};
          float d = 0.f;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            d = fmaf(bf16lo(qw[i]), bf16lo(kw[i]), d);
            d = fmaf(bf16hi(qw[i]), bf16hi(kw[i]), d);
          }
          d += __shfl_xor_sync(0xffffffffu, d, 1);
          d += __shfl_xor_sync(0xffffffffu, d, 2);
          d += __shfl_xor_sync(0xffffffffu, d, 4);
          if (q_part == 0) s_ref[r] = -d * p.scale_log2;
        }
      }
      fence_async_smem();  // the MMA reads Q through the async proxy
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(kBarQ));
      // (b) the parent array, for the walks below
      if (need_tree && !p.tree_mask && st_id < T) {
        const bool okp = st_id == 0 ? par_raw == -1 : (par_raw >= 0 && par_raw < st_id);
        s_par[st_id] = static_cast<signed char>(okp ? par_raw : -2);
      }
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kSmThreads) : "memory");
    // (c) tree visibility, transposed: bit r of s_desc[t] = query row r sees tree key t
    if (live && need_tree && st_id < n_valid) {
      const int node = (mtile * N + st_id) >> p.g_shift;
      uint64_t lo = 0, hi = 0;
      bool bad = false;
      if (p.tree_mask) {
        lo = p.tree_mask[2 * static_cast<int64_t>(node_base + node)];
        hi = p.tree_mask[2 * static_cast<int64_t>(node_base + node) + 1];
      } else {
        int u = node;
        for (int step = 0; step < T; ++step) {  // ancestor-or-self chain; a bad entry ends it
          if (u < 64) lo |= 1ull << u; else hi |= 1ull << (u - 64);
          const int pu = s_par[u];
          if (pu == -2) bad = true;
          if (pu < 0) break;
          u = pu;
        }
        if (s_par[0] == -2) bad = true;
      }
      if (bad && split == 0 && kvh == 0) dev_status_or(p.status, b, FALCON_DEV_BAD_TREE);
      if (has_tree_keys) {
        const uint32_t word = st_id >> 5, bit = 1u << (st_id & 31);
        while (lo) {
          const int t = __ffsll(static_cast<long long>(lo)) - 1;
          lo &= lo - 1;
          atomicOr(&s_desc[t * C::kDescWords + word], bit);
        }
        while (hi) {
          const int t = 64 + __ffsll(static_cast<long long>(hi)) - 1;
          hi &= hi - 1;
          atomicOr(&s_desc[t * C::kDescWords + word], bit);
        }
      }
    }
    if (has_tree_keys) asm volatile("bar.sync 1, %0;" ::"n"(kSmThreads) : "memory");
    FALCON_TRACE(tid == 64, 30);

    float neg_ref[kChunks][kCW];
#pragma unroll
    for (int ci = 0; ci < kChunks; ++ci) {
      const int ch = grp + kColGroups * ci;
#pragma unroll
      for (int c = 0; c < kCW; ++c) {
        neg_ref[ci][c] = (live && ch < n_chunks) ? s_ref[ch * kCW + c] : 0.f;
      }
    }
    const float scale = p.scale_log2;

    for (int j = 0; live && j < n_my; ++j) {
      const int sb = j & 1, st = j % kStages;
      const int k0 = key_begin + j * kBK, key = k0 + kr;
      if (!mbar_wait_warp(bar(kBarSFull + sb), (j >> 1) & 1, abort_flag)) { live = false; break; }
      FALCON_TRACE(tid == 64 && j < 4, 32 + 3 * j);
      tc_fence_after();
      uint32_t sr[kChunks][kCW];
#pragma unroll
      for (int ci = 0; ci < kChunks; ++ci) {
        const int ch = grp + kColGroups * ci;
        if (ch < n_chunks) FALCON_TMEM_LD16(tmem_lane + sb * C::kColStride + ch * kCW, sr[ci]);
      }
      tmem_wait_ld();
      FALCON_TRACE(tid == 64 && j < 4, 33 + 3 * j);

      const bool full = k0 + kBK <= Lc;  // the whole tile lies in the prefix: every key exists and is visible
      unsigned char* ptile = smem_gen + C::kOffKV + st * kStageBytes;
      if (!full && k0 + kBK > S_valid && grp == 0) {
        // The sequence's last tile: V rows past the last key may hold anything (0 x NaN = NaN in the
        // MMA).  The rows up to the next multiple of 16 are read by the last MMA step: clear them.
        if (!mbar_wait_warp(bar(kBarKVFull + st), (j / kStages) & 1, abort_flag)) { live = false; break; }
        const int nv = S_valid - k0;
        if (kr >= nv && kr < ((nv + 15) & ~15)) {
#pragma unroll
          for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int u = 0; u < 8; ++u)
              *reinterpret_cast<uint4*>(ptile + kTileBytes + h * kHalfTile + kr * 128 + u * 16) = make_uint4(0, 0, 0, 0);
        }
      }
#pragma unroll
      for (int ci = 0; ci < kChunks; ++ci) {
        const int ch = grp + kColGroups * ci;
        if (ch < n_chunks) {
          uint32_t vis = 0xffffu;
          if (!full) {
            if (key >= S_valid) vis = 0u;
            else if (key >= Lc) vis = (s_desc[(key - Lc) * C::kDescWords + (ch >> 1)] >> ((ch & 1) * 16)) & 0xffffu;
          }
          uint32_t pk[kCW / 2];
#pragma unroll
          for (int c = 0; c < kCW; c += 2) {
            float p0 = ex2(fmaf(__uint_as_float(sr[ci][c]), scale, neg_ref[ci][c]));
            float p1 = ex2(fmaf(__uint_as_float(sr[ci][c + 1]), scale, neg_ref[ci][c + 1]));
            if (!full) {
              p0 = ((vis >> c) & 1u) ? p0 : 0.f;
              p1 = ((vis >> (c + 1)) & 1u) ? p1 : 0.f;
            }
            // The weights are cut to bf16 by dropping the low half (they are positive, and the row
            // sums are taken over the same cut values as the accumulator, so the common bias cancels).
            pk[c >> 1] = __byte_perm(__float_as_uint(p0), __float_as_uint(p1), 0x7632);
          }
          // P^T row of this key: 16 query columns = two 16-byte units of the 64-column block ch / 4
          unsigned char* prow = ptile + (ch >> 2) * kHalfTile + kr * 128;
          const int u0 = 2 * (ch & 3);
          *reinterpret_cast<uint4*>(prow + ((u0 ^ (kr & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          *reinterpret_cast<uint4*>(prow + (((u0 + 1) ^ (kr & 7)) << 4)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
        }
      }
      fence_async_smem();  // the MMA reads P^T (and the cleared V rows) through the async proxy
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(kBarPFull + sb));
      FALCON_TRACE(tid == 64 && j < 4, 34 + 3 * j);
    }

    // ---- this CTA's partial result goes straight into the shared memory of the CTAs that own it ----
    // Head-dim row kr belongs to CTA kr / d_per; this split's rows have a slot there (its own rows
    // stay in the staging area).  The row sums (two bf16 rows: value and remainder) go to every CTA.
    const int o_me = kr / d_per, dl_me = kr - o_me * d_per;
    auto slot_addr = [&](int owner) -> uint32_t {  // shared::cluster address of this split's slot in `owner`
      const uint32_t local = owner == split ? smem_base + C::kOffStage
                                            : smem_base + C::kOffMrg + static_cast<uint32_t>(split < owner ? split : split - 1) * slot_bytes;
      return map_to_rank(local, static_cast<uint32_t>(owner));
    };
    bool have = live && n_my > 0 && !*abort_flag;
    if (have) have = mbar_wait_warp(bar(kBarODone), 0, abort_flag);
    FALCON_TRACE(tid == 64, 44);
    tc_fence_after();
    // Q, the ring and P^T are idle now (all of this CTA's MMAs have finished, all its loads landed).
    if (n_splits > 1) cluster_wait();  // phase 1 (arrived long ago): every peer's merge barrier is initialised
    const uint32_t row_dst = slot_addr(o_me) + static_cast<uint32_t>(dl_me) * pitch;
    const uint32_t row_bar = map_to_rank(bar(kBarMrg), static_cast<uint32_t>(o_me));
#pragma unroll
    for (int ci = 0; ci < kChunks; ++ci) {
      const int ch = grp + kColGroups * ci;
      if (ch < n_chunks) {
        uint32_t o[kCW], ls[kCW];
#pragma unroll
        for (int c = 0; c < kCW; ++c) o[c] = ls[c] = 0u;
        if (have) {
          FALCON_TMEM_LD16(tmem_lane + 2 * C::kColStride + ch * kCW, o);
          if (q4 == 0) FALCON_TMEM_LD16(tmem_lane + 3 * C::kColStride + ch * kCW, ls);
          tmem_wait_ld();
        }
        uint32_t h[kCW / 2];
#pragma unroll
        for (int c = 0; c < kCW; c += 2) {
          const __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(o[c]), __uint_as_float(o[c + 1]));
          h[c >> 1] = *reinterpret_cast<const uint32_t*>(&hh);
        }
        st_async_v4(row_dst + ch * 32, h[0], h[1], h[2], h[3], row_bar);
        st_async_v4(row_dst + ch * 32 + 16, h[4], h[5], h[6], h[7], row_bar);
        if (q4 == 0 && lane < n_splits) {
          // every TMEM lane holds the row sums: lane i of this warp sends them to CTA i
          uint32_t hv[kCW / 2], hr[kCW / 2];
#pragma unroll
          for (int c = 0; c < kCW; c += 2) {
            const float l0 = __uint_as_float(ls[c]), l1 = __uint_as_float(ls[c + 1]);
            const __nv_bfloat162 a2 = __floats2bfloat162_rn(l0, l1);
            const __nv_bfloat162 r2 = __floats2bfloat162_rn(l0 - __low2float(a2), l1 - __high2float(a2));
            hv[c >> 1] = *reinterpret_cast<const uint32_t*>(&a2);
            hr[c >> 1] = *reinterpret_cast<const uint32_t*>(&r2);
          }
          const uint32_t ldst = slot_addr(lane) + static_cast<uint32_t>(d_per) * pitch + ch * 32;
          const uint32_t lbar = map_to_rank(bar(kBarMrg), static_cast<uint32_t>(lane));
          st_async_v4(ldst, hv[0], hv[1], hv[2], hv[3], lbar);
          st_async_v4(ldst + 16, hv[4], hv[5], hv[6], hv[7], lbar);
          st_async_v4(ldst + pitch, hr[0], hr[1], hr[2], hr[3], lbar);
          st_async_v4(ldst + pitch + 16, hr[4], hr[5], hr[6], hr[7], lbar);
        }
      }
    }
    FALCON_TRACE(tid == 64, 45);
  } 
  if (warp < kWarpSm0 && n_splits > 1) cluster_wait();  // the producer and MMA warps complete phase 1 too

  // ================================ merge ================================
  // Wait until every softmax warp of every split has delivered its share of this CTA's rows.  Every
  // CTA delivers whatever happened to it, so the wait ends; it is bounded all the same.
  FALCON_TRACE(tid == 0, 50);
  bool got = mbar_wait_cluster_warp(bar(kBarMrg), 0);
  FALCON_TRACE(tid == 0, 52);
  if (tid == 0 && (*abort_flag || !got)) dev_status_or(p.status, b, FALCON_DEV_TIMEOUT);
  const unsigned char* mrg = smem_gen + C::kOffMrg;
  const unsigned char* own = smem_gen + C::kOffStage;
  // This CTA's head-dim rows summed over the splits (in split order, so the result does not depend on
  // timing), normalised and stored.  An item is one head-dim row and 4 query rows; consecutive
  // threads take consecutive head-dim rows (adjacent bf16 in `out`).  A row whose sum is too far
  // from the reference's scale (or not finite) is left to the exact path below.
  __nv_bfloat16* out_base = p.out + (static_cast<int64_t>(node_base) * p.Hq + kvh * G) * kD + d0;
  const int n_q4 = (n_valid + 3) >> 2;
  FALCON_TRACE(tid == 0, 56);
  for (int item = tid; item < d_mine * n_q4; item += kThreads) {
    const int qc = item / d_mine, dl = item - qc * d_mine;
    uint2 x[kMaxSplits], lv[kMaxSplits], lr[kMaxSplits];
#pragma unroll
    for (int s = 0; s < kMaxSplits; ++s) {
      x[s] = lv[s] = lr[s] = make_uint2(0u, 0u);
      if (s < n_splits) {
        const unsigned char* base = (s == split) ? own : mrg + static_cast<uint32_t>(s < split ? s : s - 1) * slot_bytes;
        x[s] = *reinterpret_cast<const uint2*>(base + static_cast<uint32_t>(dl) * pitch + qc * 8);
        lv[s] = *reinterpret_cast<const uint2*>(base + static_cast<uint32_t>(d_per) * pitch + qc * 8);
        lr[s] = *reinterpret_cast<const uint2*>(base + static_cast<uint32_t>(d_per + 1) * pitch + qc * 8);
      }
    }
    FALCON_TRACE(tid == 0 && x[0].x != 0x12345u, 57);
    float acc[4] = {0.f, 0.f, 0.f, 0.f}, ls[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int s = 0; s < kMaxSplits; ++s) {
      acc[0] += bf16lo(x[s].x);
      acc[1] += bf16hi(x[s].x);
      acc[2] += bf16lo(x[s].y);
      acc[3] += bf16hi(x[s].y);
      ls[0] += bf16lo(lv[s].x) + bf16lo(lr[s].x);
      ls[1] += bf16hi(lv[s].x) + bf16hi(lr[s].x);
      ls[2] += bf16lo(lv[s].y) + bf16lo(lr[s].y);
      ls[3] += bf16hi(lv[s].y) + bf16hi(lr[s].y);
    }
    FALCON_TRACE(tid == 0 && acc[0] != 1.2345f, 58);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int r = qc * 4 + c;
      if (r < n_valid) {
        if (got && ls[c] >= kLMin && ls[c] <= kLMax) {
          const int mg = mtile * N + r;
          out_base[((mg >> p.g_shift) * p.Hq + (mg & (G - 1))) * kD + dl] = __float2bfloat16_rn(__fdividef(acc[c], ls[c]));
        } else if (dl == 0) {
          s_rescue[r] = 1;
        }
      }
    }
  }
  FALCON_TRACE(tid == 0, 53);
  __syncthreads();
  // exact path for the rows that need it, shared out over the cluster's CTAs and this CTA's warps
  for (int r = split + n_splits * warp; r < n_valid; r += n_splits * (kThreads / 32))
    if (s_rescue[r]) rescue_row(p, b, kvh, node_base, T, Lc, S_valid, mtile * N + r, lane);
#ifdef FALCON_TCK_EXIT_BARRIER
  if (n_splits > 1) { cluster_arrive_relaxed(); cluster_wait(); }
#endif
  FALCON_TRACE(tid == 0, 54);
  if (warp == kWarpMma) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols) : "memory");
  }
}

bool is_pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }

template <int kChunks>
int pick_splits(falcon_ctx* ctx, int units, int max_tiles) {
  int* resident = ctx->attn_resident[kChunks];
  int best = 1;
  for (int s = kMaxSplits; s >= 1; --s) {
    if (s > max_tiles) continue;
    if (resident[s] == 0) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(s, ctx->sm_count, 1);
      cfg.blockDim = dim3(kThreads);
      cfg.dynamicSmemBytes = Cfg<kChunks>::kSmemBytes;
      cudaLaunchAttribute attr;
      attr.id = cudaLaunchAttributeClusterDimension;
      attr.val.clusterDim.x = s;
      attr.val.clusterDim.y = 1;
      attr.val.clusterDim.z = 1;
      cfg.attrs = &attr;
      cfg.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, tree_attn_tck_kernel<kChunks>, &cfg) != cudaSuccess) n = -1;
      resident[s] = n > 0 ? n : -1;
      cudaGetLastError();
    }
    if (resident[s] >= units) { best = s; break; }
  }
  return best;
}

template <int kChunks>
int launch_impl(falcon_ctx* ctx, const falcon_attn_args& a, cudaStream_t s, int q_nodes) {
  using C = Cfg<kChunks>;
  const int B = a.tree.batch, Hq = a.n_q_heads, Hkv = a.n_kv_heads, G = Hq / Hkv;
  const int N = q_nodes * G;
  const int n_units = (a.tree.max_tree + q_nodes - 1) / q_nodes;
  if (static_cast<int64_t>(Hkv) * n_units > 65535) return FALCON_ERR_CAPACITY;

  bool& attr_set = ctx->attn_attr_set[kChunks];
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(tree_attn_tck_kernel<kChunks>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(C::kSmemBytes));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaFuncSetAttribute(tree_attn_tck_kernel)");
    attr_set = true;
  }
  // Tensor maps.  The head dimension is split into (64 columns, 2 halves) so that one box covers both
  // 128-byte-swizzled half tiles.  K/V cache: [64, s_cap, 2, Hkv, B], box 64 x 128 keys x 2.
  uint64_t kv_dims[5] = {64, static_cast<uint64_t>(a.s_cap), 2, static_cast<uint64_t>(Hkv), static_cast<uint64_t>(B)};
  uint64_t kv_strides[4] = {static_cast<uint64_t>(a.kv_stride_s) * 2, 128, static_cast<uint64_t>(a.kv_stride_h) * 2,
                            static_cast<uint64_t>(a.kv_stride_b) * 2};
  if (Hkv == 1 && kv_strides[2] == 0) kv_strides[2] = kv_strides[0] * a.s_cap;  // a size-1 dimension never strides
  if (B == 1 && kv_strides[3] == 0) kv_strides[3] = kv_strides[2] * Hkv;
  const uint32_t kv_box[5] = {64, static_cast<uint32_t>(kBK), 2, 1, 1};
  CUtensorMap mk, mv;
  if (!get_tmap(ctx, a.k_cache, kv_dims, kv_strides, kv_box, &mk) || !get_tmap(ctx, a.v_cache, kv_dims, kv_strides, kv_box, &mv)) {
    ctx->last_error = "cuTensorMapEncodeTiled failed";
    return FALCON_ERR_CUDA;
  }
  const int max_tiles = (a.tree.max_prefix_len + a.tree.max_tree + kBK - 1) / kBK;
  int splits = a.n_splits;
  if (splits == 0) splits = pick_splits<kChunks>(ctx, Hkv * n_units * B, max_tiles > 0 ? max_tiles : 1);
  if (splits < 1) splits = 1;
  // every CTA must have room for the other splits' shares of the partial results
  while (splits > 1 && static_cast<uint32_t>(splits - 1) * ((kD + splits - 1) / splits + 2) * part_pitch(N) > C::kMrgBytes)
    --splits;

  TckParams p;
  p.Hq = Hq;
  p.Hkv = Hkv;
  p.G = G;
  p.g_shift = 0;
  while ((1 << p.g_shift) < G) ++p.g_shift;
  p.s_cap = a.s_cap;
  p.total_nodes = a.tree.total_nodes;
  p.n_rows = N;
  p.idesc_qk = make_idesc(kBK, N, false, false);
  p.idesc_pv = make_idesc(kD, N, true, true);
  p.idesc_sum = make_idesc(128, N, false, true);
  p.scale_log2 = a.sm_scale * kLog2e;
  p.node_off = a.tree.node_off;
  p.parent = a.tree.parent;
  p.prefix_len = a.tree.prefix_len;
  p.status = a.tree.status;
  p.tree_mask = a.tree_mask;
  p.q = static_cast<const __nv_bfloat16*>(a.q);
  p.k = static_cast<const __nv_bfloat16*>(a.k_cache);
  p.v = static_cast<const __nv_bfloat16*>(a.v_cache);
  p.kv_stride_b = a.kv_stride_b;
  p.kv_stride_h = a.kv_stride_h;
  p.kv_stride_s = a.kv_stride_s;
  p.out = static_cast<__nv_bfloat16*>(a.out);
  p.have_host = 0;
  p.early_prefix = (a.flags & FALCON_ATTN_PREFIX_STABLE) ? 1 : 0;
  if (a.tree.prefix_len_host && a.tree.node_off_host && B <= kHostSeqs) {
    p.have_host = 1;
    for (int i = 0; i <= B; ++i) p.h_node_off[i] = a.tree.node_off_host[i];
    for (int i = 0; i < B; ++i) p.h_prefix[i] = a.tree.prefix_len_host[i];
  }

  FALCON_TRACE_LAUNCH(p)

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(splits, Hkv * n_units, B);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = splits;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  cudaError_t e = cudaLaunchKernelEx(&cfg, tree_attn_tck_kernel<kChunks>, mk, mv, p);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "tree_attn_tck_kernel launch");
  return FALCON_OK;
}

}  // namespace

bool tree_attn_tck_supports(const falcon_ctx* ctx, const falcon_attn_args& a) {
  (void)ctx;
  if (a.head_dim != kD) return false;
  if (a.k_tree != nullptr) return false;
  const int G = a.n_q_heads / a.n_kv_heads;
  if (!is_pow2(G) || G > 128) return false;
  if (a.n_splits > kMaxSplits) return false;
  if (a.tree.batch > 65535) return false;
  return get_encode() != nullptr;
}

int launch_tree_attn_tck(falcon_ctx* ctx, const falcon_attn_args& a, cudaStream_t s) {
  const int G = a.n_q_heads / a.n_kv_heads;
  // Nodes per unit: as many as the tree has, in steps that make the row count a multiple of 16,
  // at most 128 rows.
  const int gran = G >= 16 ? 1 : 16 / G;
  int q_nodes = 128 / G;
  const int want = (a.tree.max_tree + gran - 1) / gran * gran;
  if (want < q_nodes) q_nodes = want;
  return q_nodes * G <= 64 ? launch_impl<1>(ctx, a, s, q_nodes) : launch_impl<2>(ctx, a, s, q_nodes);
}

}  // namespace falcon
