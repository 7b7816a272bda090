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
// (prefix + tree) into runs of whole tiles.  Each CTA owns a share of the 128 head-dim rows of the
// block's result: every CTA sends the other CTAs' shares of its partial O^T (bf16) and its row
// sums (fp32) straight from registers into their shared memory (st.async, counted on the owner's
// mbarrier), and every owner adds what it received, normalises and stores.  No partial result
// touches global memory, and there is no cluster barrier after the first.
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
//   warp 0     TMA producer: K and V tiles (up to 128 keys, 128-byte swizzle, evict-first) into a ring.
//   warp 1     one elected lane issues tcgen05.mma: S^T(j) = K(j).Q^T into one of two TMEM score
//              buffers, O^T += V(j)^T.P(j)^T with P^T read from shared memory.
//   warps 2-17 softmax: first the Q block by plain loads into the layout the MMA reads, the row
//              references and the tree's visibility sets; then, per tile, warp w works on TMEM lane
//              quadrant w % 4 (32 keys) and on the column chunks (w - 2) / 4, + 4, ... of the query
//              rows: tcgen05.ld, p = 2^(s.scale - ref), tree mask from the key's descendant bit set,
//              this key's share of the row sums in registers, P^T as bf16 into the shared memory of
//              the K tile it was computed from (free once S^T exists).
// All three falcon kernels are launched programmatically dependent; set-up that touches no global
// memory, and one prefix tile when the caller declared the prefix stable, come before
// griddepcontrol.wait.  Every mbarrier wait is bounded; a wait that runs out sets FALCON_DEV_TIMEOUT,
// what is in flight is drained, and the rows are still delivered (by the exact path).
#include <algorithm>

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
constexpr int kBKMax = 128;                     // keys per tile at most = TMEM lanes (the launcher picks the tile height)
// Three variants by the number of query rows N of a unit.  A softmax thread works on chunks of kCW
// query columns; chunk c belongs to column group c % kGroups, and a lane quadrant has one warp per
// column group.
//   0: N <= 64   4 groups, one chunk of 16 columns a thread             (18 warps)
//   1: N <= 80   5 groups, one chunk of 16 columns a thread             (22 warps)
//   2: N <= 128  4 groups, up to four chunks of 8 columns a thread, so that e.g. 96 rows spread
//                evenly; registers do not hold all chunks at once, so they are handled in turn
template <int kVar>
struct Var {
  static constexpr int kGroups = kVar == 1 ? 5 : 4;
  static constexpr int kCW = kVar == 2 ? 8 : 16;
  static constexpr int kPer = kVar == 2 ? 4 : 1;
  static constexpr int kNMax = kVar == 0 ? 64 : (kVar == 1 ? 80 : 128);
  static constexpr int kCfg = kVar == 0 ? 1 : 2;           // which Cfg (small arrays sized for 64 or 128 rows)
  static constexpr int kSmWarps = 4 * kGroups;
  static constexpr int kSmThreads = 32 * kSmWarps;
  static constexpr int kThreads = 32 * (2 + kSmWarps);     // producer, MMA issuer, softmax warps
  static constexpr int kRowsPerPass = kSmThreads / 8;      // Q rows the softmax threads load at once (8 threads a row)
  static constexpr int kQPasses = (kNMax + kRowsPerPass - 1) / kRowsPerPass;
};
constexpr int kWarpProducer = 0;
constexpr int kWarpMma = 1;
constexpr int kWarpSm0 = 2;
constexpr int kMaxSplits = 8;
constexpr int kHostSeqs = 8;
constexpr uint32_t kSmemMax = 232448;           // dynamic shared memory a CTA may ask for
constexpr float kLMin = 7.8886090522101181e-31f;  // 2^-100
constexpr float kLMax = 1.2676506002282294e+30f;  // 2^100
constexpr uint32_t kMrgSpin = 1u << 26;         // tries of the one wait that must not give up early
// Prefix tiles requested before the grid dependency wait.  One: with more, the Q block (loaded
// after the wait) queues behind them in the memory system and everything starts later (measured).
constexpr int kEarlyTiles = 1;

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

// kChunks = 1: room for 64 query rows per unit; kChunks = 2: for 128.  Shared memory, from offset 0:
// the Q block (n_rows x 256 bytes), the K/V ring (stages x tile_keys x 512 bytes), the merge area
// (what the other splits deliver), and a block of small arrays whose layout is below.  The ring
// takes what the rest leaves: the launcher picks the tile height and the number of stages.
template <int kChunks>
struct Cfg {
  static constexpr int kN = 64 * kChunks;
  static constexpr uint32_t kDescWords = kN / 32;
  static constexpr uint32_t kOffDesc = 0;                                // [128 tree keys][kN / 32] words
  static constexpr uint32_t kOffRef = kOffDesc + 128 * kDescWords * 4;   // [kN] fp32
  static constexpr uint32_t kOffLpart = kOffRef + kN * 4;                // [4][kN] fp32: the lane quadrants' shares of the row sums
  static constexpr uint32_t kOffRescue = kOffLpart + 16 * kN;            // [kN] bytes
  static constexpr uint32_t kOffPar = kOffRescue + kN;                   // [128] int8: the tree's parent array
  static constexpr uint32_t kOffBars = kOffPar + 128;
  static constexpr uint32_t kOffMisc = kOffBars + 8 * kNumBars;          // tmem base, abort flag
  static constexpr uint32_t kSmallBytes = kOffMisc + 16;
};

// bytes between the rows of a partial result of n query columns: an odd number of 16-byte units, so
// that 16-byte accesses of consecutive rows fall into different banks
__host__ __device__ constexpr uint32_t part_pitch(int n) { return static_cast<uint32_t>(n) * 2u + 16u; }

struct TckParams {
  int32_t Hq, Hkv, G, g_shift, s_cap, total_nodes;
  int32_t n_rows;          // query rows per unit (multiple of 16, at most Cfg::kN)
  int32_t tile_keys;       // keys per K/V tile (multiple of 16, at most 128)
  int32_t n_stages;        // ring depth, 2 or 3
  uint32_t off_mrg;        // shared-memory offsets of the merge area and of the small arrays
  uint32_t off_small;
  uint32_t idesc_qk, idesc_pv;
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
  int32_t stall_first;     // test hook: tile 0 is never requested (a bounded wait then runs out)
  int32_t prefetch_next;   // tm_nk / tm_nv describe the caches of the next call: bring their prefix tiles into L2
  int32_t h_node_off[kHostSeqs + 1];
  int32_t h_prefix[kHostSeqs];
  int32_t h_order[kHostSeqs];  // grid z -> sequence, longest first (CTAs are handed out in grid order: with more
                               // CTAs than SMs the long sequences must not be the ones that start last)
  FALCON_TRACE_PARAMS
};

// K/V tiles are read once per call and the caches are far larger than L2: the loads carry an
// evict-first policy, so the stream does not push out what is reused (q, the outputs, the next
// kernel's operands).
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_5d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                                 int c3, int c4, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, "
      "%6, %7}], [%2], %8;" ::"r"(dst),
      "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "l"(pol)
      : "memory");
}

__device__ __forceinline__ void prefetch_tile_l2(const CUtensorMap* map, int key0, int kvh, int b) {
  asm volatile("cp.async.bulk.prefetch.tensor.5d.L2.global.tile [%0, {%1, %2, %3, %4, %5}];" ::"l"(map), "r"(0), "r"(key0),
               "r"(0), "r"(kvh), "r"(b)
               : "memory");
}

// (d0, d1) = (a0, a1) * (b0, b1) + (c0, c1) in one instruction
__device__ __forceinline__ void fma2(float a0, float a1, float b0, float b1, float c0, float c1, float& d0, float& d1) {
  asm("{ .reg .b64 ra, rb, rc, rd; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; mov.b64 rc, {%6, %7}; "
      "fma.rn.f32x2 rd, ra, rb, rc; mov.b64 {%0, %1}, rd; }"
      : "=f"(d0), "=f"(d1)
      : "f"(a0), "f"(a1), "f"(b0), "f"(b1), "f"(c0), "f"(c1));
}
// (x0, x1) += (y0, y1) in one instruction
__device__ __forceinline__ void add2(float& x0, float& x1, float y0, float y1) {
  asm("{ .reg .b64 ra, rb, rd; mov.b64 ra, {%0, %1}; mov.b64 rb, {%2, %3}; add.rn.f32x2 rd, ra, rb; mov.b64 {%0, %1}, rd; }"
      : "+f"(x0), "+f"(x1)
      : "f"(y0), "f"(y1));
}
template <int kW>
__device__ __forceinline__ void tmem_ld_chunk(uint32_t taddr, uint32_t (&r)[kW]) {
  if constexpr (kW == 16) {
    FALCON_TMEM_LD16(taddr, r);
  } else {
    static_assert(kW == 8, "chunk width");
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
  }
}

// 16 bytes into the shared memory of a CTA of the cluster (this one included); the store counts 16
// bytes on the mbarrier `bar`, which must live in the same CTA as the destination.
__device__ __forceinline__ void st_async_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(addr),
               "r"(a), "r"(b), "r"(c), "r"(d), "r"(bar)
               : "memory");
}
// Bounded wait of one thread that does not look at the CTA's abort flag: for draining what is in
// flight after another wait has given up.
__device__ __forceinline__ bool mbar_wait_drain(uint32_t bar, uint32_t parity) {
  for (uint32_t it = 0; it < (1u << 20); ++it) {
    uint32_t ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok)
                 : "r"(bar), "r"(parity)
                 : "memory");
    if (ok) return true;
  }
  return false;
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

// Sums over the warp's lanes of v[c] for each of kW columns (a fixed order of additions); lane L
// ends with the sum of column col_of_lane<kW>(L).
template <int kW>
__device__ __forceinline__ float warp_col_sums(const float (&v)[kW], int lane) {
  float a[8];
  if constexpr (kW == 16) {
    const bool hi = lane & 16;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float send = hi ? v[i] : v[i + 8], keep = hi ? v[i + 8] : v[i];
      a[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) a[i] = v[i] + __shfl_xor_sync(0xffffffffu, v[i], 16);
  }
  float b4[4], c2[2];
  {
    const bool hi = lane & 8;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float send = hi ? a[i] : a[i + 4], keep = hi ? a[i + 4] : a[i];
      b4[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
    }
  }
  {
    const bool hi = lane & 4;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const float send = hi ? b4[i] : b4[i + 2], keep = hi ? b4[i + 2] : b4[i];
      c2[i] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    }
  }
  const bool hi = lane & 2;
  const float send = hi ? c2[0] : c2[1], keep = hi ? c2[1] : c2[0];
  float d = keep + __shfl_xor_sync(0xffffffffu, send, 2);
  d += __shfl_xor_sync(0xffffffffu, d, 1);
  return d;
}
template <int kW>
__device__ __forceinline__ int col_of_lane(int lane) {
  return (kW == 16 ? ((lane >> 4) & 1) * 8 : 0) + ((lane >> 3) & 1) * 4 + ((lane >> 2) & 1) * 2 + ((lane >> 1) & 1);
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

// kFull: the ring is three stages of 128-key tiles (then the geometry is known at compile time).
template <int kVar, bool kFull>
__global__ void __launch_bounds__(Var<kVar>::kThreads, 1)
tree_attn_tck_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                     const __grid_constant__ CUtensorMap tm_nk, const __grid_constant__ CUtensorMap tm_nv,
                     const TckParams p) {
  using VT = Var<kVar>;
  using C = Cfg<VT::kCfg>;
  constexpr int kColGroups = VT::kGroups, kSmWarps = VT::kSmWarps, kSmThreads = VT::kSmThreads, kThreads = VT::kThreads;
  extern __shared__ __align__(1024) unsigned char smem_gen[];
  const uint32_t smem_base = smem_u32(smem_gen);
  unsigned char* small = smem_gen + p.off_small;
  uint32_t* s_desc = reinterpret_cast<uint32_t*>(small + C::kOffDesc);
  float* s_ref = reinterpret_cast<float*>(small + C::kOffRef);
  unsigned char* s_rescue = small + C::kOffRescue;
  signed char* s_par = reinterpret_cast<signed char*>(small + C::kOffPar);
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(small + C::kOffMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(small + C::kOffMisc + 4);
  const uint32_t bars = smem_base + p.off_small + C::kOffBars;
  // K/V ring geometry
  const int BK = kFull ? kBKMax : p.tile_keys, kStages = kFull ? 3 : p.n_stages;
  const uint32_t kHalfTile = static_cast<uint32_t>(BK) * 128u;   // one 64-column half of a K or V tile
  const uint32_t kTileBytes = 2u * kHalfTile, kStageBytes = 2u * kTileBytes;
  const uint32_t off_q = 0, off_kv = static_cast<uint32_t>(p.n_rows) * 256u, off_mrg = p.off_mrg, off_stage = 0;
  const uint32_t tmem_cols = (kVar == 0 || p.n_rows <= 64) ? 256u : 512u, col_stride = tmem_cols / 4;  // S^T(0), S^T(1), O^T
  auto bar = [&](int i) { return bars + 8u * static_cast<uint32_t>(i); };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_splits = gridDim.x, split = blockIdx.x;  // cluster = all CTAs of a row of the grid
  const int kvh = blockIdx.y % p.Hkv, mtile = blockIdx.y / p.Hkv;
  const int b = p.have_host ? p.h_order[blockIdx.z] : static_cast<int>(blockIdx.z);
  constexpr int kCW = VT::kCW, kPer = VT::kPer;
  const int G = p.G, N = p.n_rows, n_chunks = N / kCW;
  const uint32_t q_half_bytes = static_cast<uint32_t>(N) * 128u;  // between the two 64-column halves of Q
  FALCON_TRACE(tid == 0, 0);
  if (warp == kWarpProducer) {
    // the barriers first: their initialisation (and its fence) runs under the parameter reads below
    if (lane == 0) {
      *abort_flag = (smem_base & 1023u) ? 1 : 0;  // the swizzled tiles need a 1 KB aligned base
      prefetch_tmap(&tm_k);
      prefetch_tmap(&tm_v);
    }
    if (lane < kNumBars)
      mbar_init(bar(lane), (lane == kBarPFull || lane == kBarPFull + 1 || lane == kBarQ) ? kSmWarps : 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
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
  FALCON_TRACE(tid == 0, 20);

  // Geometry of this CTA's share, from the sequence's node range and prefix length.
  int node_base = 0, T_real = 0, L_raw = 0;
  int T = 0, rows_total, n_valid = 0, L = 0, Lc = 0, S_valid = 0, tile_begin, tile_end = 0, n_my = 0, key_begin = 0;
  auto geometry = [&]() {
    T = min(T_real, FALCON_T_MAX);
    rows_total = T * G;
    n_valid = min(N, rows_total - mtile * N);
    L = max(L_raw, 0);
    Lc = min(L, p.s_cap);
    S_valid = min(L + T, p.s_cap);  // keys that exist below the cache capacity
    // Whole tiles per split, boundaries rounded up: a longer run goes to an early split; the last
    // one has the tree's tiles and the longest set-up (the tree's visibility sets).
    const int n_tiles = (S_valid + BK - 1) / BK;
    tile_begin = (split * n_tiles + n_splits - 1) / n_splits;
    tile_end = ((split + 1) * n_tiles + n_splits - 1) / n_splits;
    n_my = tile_end - tile_begin;
    key_begin = tile_begin * BK;
  };
  auto device_scalars = [&]() {
    node_base = p.node_off[b];
    T_real = p.node_off[b + 1] - node_base;
    L_raw = p.prefix_len[b];
    geometry();
  };
  const uint64_t kv_policy = policy_evict_first();
  auto load_tile = [&](int j) {
    if (j == 0 && p.stall_first) return;
    const int st = j % kStages;
    const uint32_t dst = smem_base + off_kv + st * kStageBytes;
    mbar_expect_tx(bar(kBarKVFull + st), kStageBytes);
    tma_load_5d_hint(dst, &tm_k, bar(kBarKVFull + st), 0, key_begin + j * BK, 0, kvh, b, kv_policy);
    tma_load_5d_hint(dst + kTileBytes, &tm_v, bar(kBarKVFull + st), 0, key_begin + j * BK, 0, kvh, b, kv_policy);
  };
  // This thread's piece of the Q block (softmax threads): 16 head-dim columns of one or two rows.
  const int st_id = tid - 32 * kWarpSm0;
  const int q_part = st_id & 7;
  auto q_piece = [&](int r) -> const __nv_bfloat16* {
    const int mg = mtile * N + r;
    return p.q + (static_cast<int64_t>(node_base + (mg >> p.g_shift)) * p.Hq + kvh * G + (mg & (G - 1))) * kD + q_part * 16;
  };
  if (p.have_host) {  // the caller's host copies of the per-sequence scalars: no round trip to global memory
    node_base = p.h_node_off[b];
    T_real = p.h_node_off[b + 1] - node_base;
    L_raw = p.h_prefix[b];
    geometry();
  }
  FALCON_TRACE(tid == 0, 22);

  // Under programmatic dependent launch the kernel starts while the previous kernel of the stream
  // is finishing; griddepcontrol.wait returns once that kernel has completed.  Each warp role waits
  // where it must: the softmax warps at once, because the loads everything waits for (Q, the
  // reference key, the tree) are theirs and their set-up can run under those loads; the producer
  // and the MMA warp after set-up that touches no global memory.
  uint4 qreg[VT::kQPasses][2], kref[2];
  int par_raw = -1;
  int n_early = 0;  // K/V tiles requested before the producer's wait
  if (warp >= kWarpSm0) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (!p.have_host) device_scalars();
    if (n_valid > 0 && n_my > 0) {
      // Q by plain loads (a TMA request would queue behind the K/V tiles already asked for), the
      // reference key (cache row 0) and the tree's parent array
#pragma unroll
      for (int pass = 0; pass < VT::kQPasses; ++pass) {
        const int r = (st_id >> 3) + VT::kRowsPerPass * pass;
        qreg[pass][0] = qreg[pass][1] = make_uint4(0u, 0u, 0u, 0u);
        if (r < n_valid) {
          qreg[pass][0] = reinterpret_cast<const uint4*>(q_piece(r))[0];
          qreg[pass][1] = reinterpret_cast<const uint4*>(q_piece(r))[1];
        }
      }
      const __nv_bfloat16* k0p = p.k + b * p.kv_stride_b + kvh * p.kv_stride_h + q_part * 16;
      kref[0] = reinterpret_cast<const uint4*>(k0p)[0];
      kref[1] = reinterpret_cast<const uint4*>(k0p)[1];
      const bool tree_here = tile_end * BK > Lc || (split == 0 && kvh == 0);
      if (tree_here && !p.tree_mask && st_id < T) par_raw = p.parent[node_base + st_id];
    }
    for (int i = st_id; i < 128 * static_cast<int>(C::kDescWords); i += kSmThreads) s_desc[i] = 0u;
    if (st_id < C::kN) s_rescue[st_id] = 0;
  } else if (warp == kWarpProducer) {
    __syncwarp();
    FALCON_TRACE(tid == 0, 21);
    if (p.have_host && n_valid > 0 && lane == 0 && p.early_prefix) {
      // Prefix rows that the caller declares stable (written before the kernel that precedes this
      // one in the stream started) may be requested while that kernel is still finishing.
      // (One tile: more would only delay the Q block, which queues behind them in the memory system.)
      const int n_ask = min(n_my, kEarlyTiles);
      for (int j = 0; j < n_ask && key_begin + (j + 1) * BK <= Lc; ++j) {
        load_tile(j);
        ++n_early;
      }
    }
    FALCON_TRACE(tid == 0, 1);
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    FALCON_TRACE(tid == 0, 2);
    if (!p.have_host) device_scalars();
  } else {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem_base)),
                 "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (!p.have_host) device_scalars();
  }
  if (n_valid <= 0) {  // no query rows here; same decision in every warp and every CTA of the cluster
    tc_fence_before();
    __syncthreads();
    if (warp == kWarpMma) {
      tc_fence_after();
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(*s_tmem_base), "r"(tmem_cols)
                   : "memory");
    }
    return;
  }
  const bool has_tree_keys = tile_end * BK > Lc;
  const bool need_tree = has_tree_keys || (split == 0 && kvh == 0);  // the latter reports malformed trees

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
      bool ok = true;
      int issued = min(n_my, kStages);
      for (int j = kStages; ok && j < n_my; ++j) {
        ok = mbar_wait(bar(kBarKVEmpty + j % kStages), (j / kStages - 1) & 1, abort_flag);
        if (ok) {
          load_tile(j);
          issued = j + 1;
        }
      }
      if (!ok || *abort_flag) {
        // Some wait gave up.  The tiles asked for still arrive: stay until they have, so that no copy
        // is in flight into this CTA's shared memory when it leaves.
        for (int j = max(0, issued - kStages); j < issued; ++j)
          if (!(j == 0 && p.stall_first)) mbar_wait_drain(bar(kBarKVFull + j % kStages), (j / kStages) & 1);
      }
      if (p.prefetch_next && ok && n_my > 0 && n_my <= kStages) {
        // The caller named the caches of the next call.  Where a CTA's whole key range fits the ring
        // (short prefixes: the loads are over early and memory idles during the rest of the
        // launch), once its last tile has landed it asks for the same tiles of those caches, as far
        // as they lie in the prefix, to be brought into L2.  With longer ranges the memory system is
        // busy to the end and a prefetch would only compete with the other CTAs' loads.
        const int jl = n_my - 1;
        if (mbar_wait(bar(kBarKVFull + jl % kStages), (jl / kStages) & 1, abort_flag)) {
          for (int j = 0; j < n_my && key_begin + (j + 1) * BK <= Lc; ++j) {
            prefetch_tile_l2(&tm_nk, key_begin + j * BK, kvh, b);
            prefetch_tile_l2(&tm_nv, key_begin + j * BK, kvh, b);
          }
        }
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
        const uint32_t kbase = smem_base + off_kv + st * kStageBytes;
        if (elected) {
#pragma unroll
          for (int kk = 0; kk < kD / 16; ++kk) {
            // K tile (A) and Q block (B): K-major, 16 head-dim columns = 32 bytes inside the 128-byte swizzle row
            const uint64_t ad = smem_desc(kbase + (kk >> 2) * kHalfTile + (kk & 3) * 32, 16, 1024);
            const uint64_t bd = smem_desc(smem_base + off_q + (kk >> 2) * q_half_bytes + (kk & 3) * 32, 16, 1024);
            umma_bf16_ss(tmem_base + sb * col_stride, ad, bd, p.idesc_qk, kk > 0 ? 1u : 0u);
          }
          umma_commit(bar(kBarSFull + sb));
          FALCON_TRACE(j == 0, 28);
        }
        __syncwarp();
        return true;
      };
      auto issue_pv = [&](int t) {
        const int st = t % kStages;
        const uint32_t pbase = smem_base + off_kv + st * kStageBytes;   // P^T lies over the K tile
        const uint32_t vbase = pbase + kTileBytes;
        // keys of the tile that exist, in MMA steps of 16 (rows above them hold zeros in P^T and V)
        const int nk = (min(BK, S_valid - (key_begin + t * BK)) + 15) >> 4;
        if (elected) {
          for (int kk = 0; kk < nk; ++kk) {
            // V^T (A) and P^T (B): both with the M / N index contiguous; 16 keys = 2 KB, the 64-column
            // blocks of either operand 16 KB apart
            const uint64_t ad = smem_desc(vbase + kk * 2048, kHalfTile, 1024);
            const uint64_t bd = smem_desc(pbase + kk * 2048, kHalfTile, 1024);
            umma_bf16_ss(tmem_base + 2 * col_stride, ad, bd, p.idesc_pv, (t > 0 || kk > 0) ? 1u : 0u);
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

    FALCON_TRACE(tid == 64 && live && qreg[0][0].x != 0x12345u, 6);
    FALCON_TRACE(tid == 64 && live && kref[0].x != 0x12345u, 7);
    FALCON_TRACE(tid == 64 && live && par_raw != 0x12345, 8);
    if (live) {
      // (a) Q block into shared memory in the layout the MMA reads (K-major rows of 128 bytes per
      // 64-column half, 16-byte units XOR-swizzled by the row).  The MMA warp is told at once; the
      // references below need cache row 0 as well, which arrives later, and nobody waits for them yet.
#pragma unroll
      for (int pass = 0; pass < VT::kQPasses; ++pass) {
        const int r = (st_id >> 3) + VT::kRowsPerPass * pass;
        if (r < N) {
          unsigned char* qrow = smem_gen + off_q + (q_part >> 2) * q_half_bytes + r * 128;
          const int u0 = 2 * (q_part & 3);
          *reinterpret_cast<uint4*>(qrow + ((u0 ^ (r & 7)) << 4)) = qreg[pass][0];
          *reinterpret_cast<uint4*>(qrow + (((u0 + 1) ^ (r & 7)) << 4)) = qreg[pass][1];
        }
      }
      fence_async_smem();  // the MMA reads Q through the async proxy
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(kBarQ));
      FALCON_TRACE(tid == 64, 9);
      // the reference of every query row: its scaled score against cache row 0 (8 threads per row,
      // 16 columns each)
      const uint32_t kw[8] = {kref[0].x, kref[0].y, kref[0].z, kref[0].w, kref[1].x, kref[1].y, kref[1].z, kref[1].w};
#pragma unroll
      for (int pass = 0; pass < VT::kQPasses; ++pass) {
        const int r = (st_id >> 3) + VT::kRowsPerPass * pass;
        if (r < N) {
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

    // The references of this thread's columns stay in registers when it has one chunk; with several
    // chunks they are read from shared memory where they are used (registers go to the row sums).
    constexpr bool kRefInRegs = kPer == 1;
    float neg_ref[kRefInRegs ? kPer : 1][kCW], l_acc[kPer][kCW];  // l_acc: this key lane's share of the row sums
#pragma unroll
    for (int ci = 0; ci < kPer; ++ci) {
      const int ch = grp + kColGroups * ci;
#pragma unroll
      for (int c = 0; c < kCW; ++c) {
        if (kRefInRegs) neg_ref[ci][c] = (live && ch < n_chunks) ? s_ref[ch * kCW + c] : 0.f;
        l_acc[ci][c] = 0.f;
      }
    }
    const float scale = p.scale_log2;

    for (int j = 0; live && j < n_my; ++j) {
      const int sb = j & 1, st = j % kStages;
      const int k0 = key_begin + j * BK, key = k0 + kr;
      if (!mbar_wait_warp(bar(kBarSFull + sb), (j >> 1) & 1, abort_flag)) { live = false; break; }
      FALCON_TRACE(tid == 64 && j < 4, 32 + 3 * j);
      tc_fence_after();
      if (q4 * 32 < BK) {  // (a tile lower than 128 keys leaves the last quadrants without keys)
      uint32_t sr[kRefInRegs ? kPer : 1][kCW];
      if (kRefInRegs) {
#pragma unroll
        for (int ci = 0; ci < kPer; ++ci) {
          const int ch = grp + kColGroups * ci;
          if (ch < n_chunks) tmem_ld_chunk<kCW>(tmem_lane + sb * col_stride + ch * kCW, sr[ci]);
        }
        tmem_wait_ld();
      }
      FALCON_TRACE(tid == 64 && j < 4, 33 + 3 * j);

      // all of this warp's keys lie in the prefix: every one exists and is visible to every row
      const bool full = k0 + BK <= Lc && q4 * 32 + 32 <= BK;
      unsigned char* ptile = smem_gen + off_kv + st * kStageBytes;
      if (!full && k0 + BK > S_valid && grp == 0) {
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
      for (int ci = 0; ci < kPer; ++ci) {
        const int ch = grp + kColGroups * ci;
        if (ch < n_chunks) {
          uint32_t vis = (1u << kCW) - 1u;
          if (!full) {
            if (key >= S_valid || kr >= BK) vis = 0u;
            else if (key >= Lc) vis &= s_desc[(key - Lc) * C::kDescWords + ((ch * kCW) >> 5)] >> ((ch * kCW) & 31);
          }
          constexpr int kSel = kRefInRegs ? 1 : 0;
          const int cr = ci * kSel;  // where this chunk's scores and references are
          if (!kRefInRegs) {  // this chunk's scores and references now (one chunk's worth of registers)
            tmem_ld_chunk<kCW>(tmem_lane + sb * col_stride + ch * kCW, sr[0]);
#pragma unroll
            for (int c = 0; c < kCW; c += 4) {
              const float4 r4 = *reinterpret_cast<const float4*>(s_ref + ch * kCW + c);
              neg_ref[0][c] = r4.x;
              neg_ref[0][c + 1] = r4.y;
              neg_ref[0][c + 2] = r4.z;
              neg_ref[0][c + 3] = r4.w;
            }
            tmem_wait_ld();
          }
          uint32_t pk[kCW / 2];
#pragma unroll
          for (int c = 0; c < kCW; c += 2) {
            // two columns at a time: one packed fma for the exponents, one packed add for the row sums
            float e0, e1;
            fma2(__uint_as_float(sr[cr][c]), __uint_as_float(sr[cr][c + 1]), scale, scale, neg_ref[cr][c], neg_ref[cr][c + 1],
                 e0, e1);
            float p0 = ex2(e0), p1 = ex2(e1);
            if (!full) {
              p0 = ((vis >> c) & 1u) ? p0 : 0.f;
              p1 = ((vis >> (c + 1)) & 1u) ? p1 : 0.f;
            }
            // The weights are cut to bf16 by dropping the low half (they are positive, and the row
            // sums take the same cut values as the accumulator, so the common bias cancels and a row
            // that one key dominates is exact whatever that key's weight is).
            const uint32_t b0 = __float_as_uint(p0), b1 = __float_as_uint(p1);
            pk[c >> 1] = __byte_perm(b0, b1, 0x7632);
            add2(l_acc[ci][c], l_acc[ci][c + 1], __uint_as_float(b0 & 0xffff0000u), __uint_as_float(b1 & 0xffff0000u));
          }
          // P^T row of this key: the chunk's columns are 16-byte units (8 columns each) of the
          // 64-column block they fall in, swizzled by the row like everything the MMA reads
          unsigned char* prow = ptile + ((ch * kCW) >> 6) * kHalfTile + kr * 128;
          const int u0 = ((ch * kCW) >> 3) & 7;
          if (kr < BK) {
#pragma unroll
            for (int u = 0; u < kCW / 8; ++u)
              *reinterpret_cast<uint4*>(prow + (((u0 + u) ^ (kr & 7)) << 4)) =
                  make_uint4(pk[4 * u], pk[4 * u + 1], pk[4 * u + 2], pk[4 * u + 3]);
          }
        }
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
    // stay in the staging area).  The row sums (fp32, in the space of two more rows) go to every CTA.
    const int o_me = kr / d_per, dl_me = kr - o_me * d_per;
    auto slot_addr = [&](int owner) -> uint32_t {  // shared::cluster address of this split's slot in `owner`
      const uint32_t local = owner == split ? smem_base + off_stage
                                            : smem_base + off_mrg + static_cast<uint32_t>(split < owner ? split : split - 1) * slot_bytes;
      return map_to_rank(local, static_cast<uint32_t>(owner));
    };
    const bool have = live && n_my > 0 && !*abort_flag;
    uint32_t own_l[4] = {0u, 0u, 0u, 0u};
    if (n_splits > 1) cluster_wait();  // phase 1 (arrived long ago): every peer's merge barrier is initialised
    // The row sums first: they are complete with the last tile's softmax pass and do not have to wait for the
    // MMAs that are still running.  They go to the other CTAs at once; this CTA's own slot lies over Q and,
    // where it is larger than Q, over the ring's first stage, which the last MMAs may still be reading: its
    // copy of the sums is written with the rest of the slot, after them.
    float* s_lpart = reinterpret_cast<float*>(small + C::kOffLpart);
#pragma unroll
    for (int ci = 0; ci < kPer; ++ci) {
      const int ch = grp + kColGroups * ci;
      if (ch < n_chunks) {
        // this warp's 32 keys' share of the chunk's row sums
        const float sum = warp_col_sums<kCW>(l_acc[ci], lane);
        if ((lane & (kCW == 16 ? 1 : 17)) == 0) s_lpart[q4 * C::kN + ch * kCW + col_of_lane<kCW>(lane)] = have ? sum : 0.f;
      }
    }
    // the four lane quadrants' shares added (fixed order), four rows per thread, to every CTA (fp32, 4 bytes a
    // query row, in the space of two more rows of the slot)
    asm volatile("bar.sync 1, %0;" ::"n"(kSmThreads) : "memory");
    if (st_id * 4 < N) {
      const float4 s0 = reinterpret_cast<const float4*>(s_lpart)[st_id];
      const float4 s1 = reinterpret_cast<const float4*>(s_lpart + C::kN)[st_id];
      const float4 s2 = reinterpret_cast<const float4*>(s_lpart + 2 * C::kN)[st_id];
      const float4 s3 = reinterpret_cast<const float4*>(s_lpart + 3 * C::kN)[st_id];
      const uint32_t l0 = __float_as_uint((s0.x + s1.x) + (s2.x + s3.x)), l1 = __float_as_uint((s0.y + s1.y) + (s2.y + s3.y));
      const uint32_t l2 = __float_as_uint((s0.z + s1.z) + (s2.z + s3.z)), l3 = __float_as_uint((s0.w + s1.w) + (s2.w + s3.w));
      for (int i = 0; i < n_splits; ++i)
        if (i != split)
          st_async_v4(slot_addr(i) + static_cast<uint32_t>(d_per) * pitch + st_id * 16, l0, l1, l2, l3,
                      map_to_rank(bar(kBarMrg), static_cast<uint32_t>(i)));
      own_l[0] = l0;
      own_l[1] = l1;
      own_l[2] = l2;
      own_l[3] = l3;
    }
    // Then O^T, once every MMA has finished.  A split whose last commit never shows up sends NaN: the owner
    // then recomputes the row on the exact path instead of dividing a short numerator by a full row sum.
    bool have_o = have;
    if (have_o) have_o = mbar_wait_warp(bar(kBarODone), 0, abort_flag);
    FALCON_TRACE(tid == 64, 44);
    tc_fence_after();
    // The ring and P^T are idle now (all of this CTA's MMAs have finished, all its loads landed).
    if (st_id * 4 < N)
      st_async_v4(slot_addr(split) + static_cast<uint32_t>(d_per) * pitch + st_id * 16, own_l[0], own_l[1], own_l[2], own_l[3],
                  map_to_rank(bar(kBarMrg), static_cast<uint32_t>(split)));
    const uint32_t row_dst = slot_addr(o_me) + static_cast<uint32_t>(dl_me) * pitch;
    const uint32_t row_bar = map_to_rank(bar(kBarMrg), static_cast<uint32_t>(o_me));
#pragma unroll
    for (int ci = 0; ci < kPer; ++ci) {
      const int ch = grp + kColGroups * ci;
      if (ch < n_chunks) {
        uint32_t o[kCW];
#pragma unroll
        for (int c = 0; c < kCW; ++c) o[c] = have ? 0x7fc00000u : 0u;
        if (have_o) {
          tmem_ld_chunk<kCW>(tmem_lane + 2 * col_stride + ch * kCW, o);
          tmem_wait_ld();
        }
        uint32_t h[kCW / 2];
#pragma unroll
        for (int c = 0; c < kCW; c += 2) {
          const __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(o[c]), __uint_as_float(o[c + 1]));
          h[c >> 1] = *reinterpret_cast<const uint32_t*>(&hh);
        }
#pragma unroll
        for (int u = 0; u < kCW / 8; ++u)
          st_async_v4(row_dst + ch * (kCW * 2) + u * 16, h[4 * u], h[4 * u + 1], h[4 * u + 2], h[4 * u + 3], row_bar);
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
  const unsigned char* mrg = smem_gen + off_mrg;
  const unsigned char* own = smem_gen + off_stage;
  // This CTA's head-dim rows summed over the splits (in split order, so the result does not depend on
  // timing), normalised and stored.  An item is one head-dim row and 4 query rows; consecutive
  // threads take consecutive head-dim rows (adjacent bf16 in `out`).  A row whose sum is too far
  // from the reference's scale (or not finite) is left to the exact path below.
  __nv_bfloat16* out_base = p.out + (static_cast<int64_t>(node_base) * p.Hq + kvh * G) * kD + d0;
  const int n_q4 = (n_valid + 3) >> 2;
  FALCON_TRACE(tid == 0, 56);
  for (int item = tid; item < d_mine * n_q4; item += kThreads) {
    const int qc = item / d_mine, dl = item - qc * d_mine;
    float acc[4] = {0.f, 0.f, 0.f, 0.f}, ls[4] = {0.f, 0.f, 0.f, 0.f};
    for (int s = 0; s < n_splits; ++s) {
      const unsigned char* base = (s == split) ? own : mrg + static_cast<uint32_t>(s < split ? s : s - 1) * slot_bytes;
      const uint2 x = *reinterpret_cast<const uint2*>(base + static_cast<uint32_t>(dl) * pitch + qc * 8);
      const float4 lv = *reinterpret_cast<const float4*>(base + static_cast<uint32_t>(d_per) * pitch + qc * 16);
      acc[0] += bf16lo(x.x);
      acc[1] += bf16hi(x.x);
      acc[2] += bf16lo(x.y);
      acc[3] += bf16hi(x.y);
      ls[0] += lv.x;
      ls[1] += lv.y;
      ls[2] += lv.z;
      ls[3] += lv.w;
    }
    FALCON_TRACE(tid == 0 && acc[0] != 1.2345f, 58);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int r = qc * 4 + c;
      if (r < n_valid) {
        if (got && ls[c] >= kLMin && ls[c] <= kLMax && acc[c] == acc[c]) {
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
  FALCON_TRACE(tid == 0, 54);
  if (warp == kWarpMma) {
    // (after a wait that gave up, MMAs may still be running: the last commit covers them all)
    if (n_my > 0 && *abort_flag && lane == 0) mbar_wait_drain(bar(kBarODone), 0);
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

bool is_pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }

template <int kVar>
int pick_splits(falcon_ctx* ctx, int units, int max_tiles) {
  int* resident = ctx->attn_resident[1 + kVar];
  int best = 1;
  for (int s = kMaxSplits; s >= 1; --s) {
    if (s > max_tiles) continue;
    if (resident[s] == 0) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(s, ctx->sm_count, 1);
      cfg.blockDim = dim3(Var<kVar>::kThreads);
      cfg.dynamicSmemBytes = kSmemMax;
      cudaLaunchAttribute attr;
      attr.id = cudaLaunchAttributeClusterDimension;
      attr.val.clusterDim.x = s;
      attr.val.clusterDim.y = 1;
      attr.val.clusterDim.z = 1;
      cfg.attrs = &attr;
      cfg.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, tree_attn_tck_kernel<kVar, true>, &cfg) != cudaSuccess) n = -1;
      resident[s] = n > 0 ? n : -1;
      cudaGetLastError();
    }
    if (resident[s] >= units) { best = s; break; }
  }
  return best;
}

template <int kVar>
int launch_impl(falcon_ctx* ctx, const falcon_attn_args& a, cudaStream_t s, int q_nodes) {
  using C = Cfg<Var<kVar>::kCfg>;
  const int B = a.tree.batch, Hq = a.n_q_heads, Hkv = a.n_kv_heads, G = Hq / Hkv;
  const int N = q_nodes * G;
  const int n_units = (a.tree.max_tree + q_nodes - 1) / q_nodes;
  if (static_cast<int64_t>(Hkv) * n_units > 65535) return FALCON_ERR_CAPACITY;

  bool& attr_set = ctx->attn_attr_set[1 + kVar];
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(tree_attn_tck_kernel<kVar, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(kSmemMax));
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(tree_attn_tck_kernel<kVar, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               static_cast<int>(kSmemMax));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaFuncSetAttribute(tree_attn_tck_kernel)");
    attr_set = true;
  }
  const int max_tiles = (a.tree.max_prefix_len + a.tree.max_tree + kBKMax - 1) / kBKMax;
  int splits = a.n_splits;
  if (splits == 0) splits = pick_splits<kVar>(ctx, Hkv * n_units * B, max_tiles > 0 ? max_tiles : 1);
  if (splits < 1) splits = 1;
  // Shared memory: Q, merge area (the other splits' shares of this CTA's head-dim rows and the row
  // sums) and the small arrays are fixed by the shape; the K/V ring takes the rest, as three stages
  // of the highest tile that fits (two if three would be lower than 64 keys).  A split count whose
  // merge area would leave less than two 64-key stages is reduced.
  const uint32_t q_bytes = static_cast<uint32_t>(N) * 256u;
  auto merge_bytes = [&](int ns) {
    return ns > 1 ? static_cast<uint32_t>(ns - 1) * ((kD + ns - 1) / ns + 2) * part_pitch(N) : 0u;
  };
  auto ring_room = [&](int ns) { return static_cast<int>(kSmemMax) - static_cast<int>(q_bytes + merge_bytes(ns) + C::kSmallBytes); };
  while (splits > 1 && ring_room(splits) < 2 * 64 * 512) --splits;
  const int room = ring_room(splits);
  int n_stages = 3, tile_keys = room / (3 * 512) / 16 * 16;
  if (tile_keys < 64) {
    n_stages = 2;
    tile_keys = room / (2 * 512) / 16 * 16;
  }
  if (tile_keys > kBKMax) tile_keys = kBKMax;
  const uint32_t off_mrg = q_bytes + static_cast<uint32_t>(n_stages * tile_keys) * 512u;
  const uint32_t off_small = off_mrg + merge_bytes(splits);
  const uint32_t smem_bytes = off_small + C::kSmallBytes;

  // Tensor maps.  The head dimension is split into (64 columns, 2 halves) so that one box covers both
  // 128-byte-swizzled half tiles.  K/V cache: [64, s_cap, 2, Hkv, B], box 64 x tile_keys x 2.
  uint64_t kv_dims[5] = {64, static_cast<uint64_t>(a.s_cap), 2, static_cast<uint64_t>(Hkv), static_cast<uint64_t>(B)};
  uint64_t kv_strides[4] = {static_cast<uint64_t>(a.kv_stride_s) * 2, 128, static_cast<uint64_t>(a.kv_stride_h) * 2,
                            static_cast<uint64_t>(a.kv_stride_b) * 2};
  if (Hkv == 1 && kv_strides[2] == 0) kv_strides[2] = kv_strides[0] * a.s_cap;  // a size-1 dimension never strides
  if (B == 1 && kv_strides[3] == 0) kv_strides[3] = kv_strides[2] * Hkv;
  const uint32_t kv_box[5] = {64, static_cast<uint32_t>(tile_keys), 2, 1, 1};
  CUtensorMap mk, mv;
  if (!get_tmap(ctx, a.k_cache, kv_dims, kv_strides, kv_box, &mk) || !get_tmap(ctx, a.v_cache, kv_dims, kv_strides, kv_box, &mv)) {
    ctx->last_error = "cuTensorMapEncodeTiled failed";
    return FALCON_ERR_CUDA;
  }
  // the next call's caches (a prefetch hint): same geometry, only with the stable-prefix promise
  CUtensorMap mnk = mk, mnv = mv;
  const bool prefetch_next = a.next_k_cache && a.next_v_cache && (a.flags & FALCON_ATTN_PREFIX_STABLE) &&
                             !((reinterpret_cast<uintptr_t>(a.next_k_cache) | reinterpret_cast<uintptr_t>(a.next_v_cache)) & 15) &&
                             get_tmap(ctx, a.next_k_cache, kv_dims, kv_strides, kv_box, &mnk) &&
                             get_tmap(ctx, a.next_v_cache, kv_dims, kv_strides, kv_box, &mnv);

  TckParams p;
  p.Hq = Hq;
  p.Hkv = Hkv;
  p.G = G;
  p.g_shift = 0;
  while ((1 << p.g_shift) < G) ++p.g_shift;
  p.s_cap = a.s_cap;
  p.total_nodes = a.tree.total_nodes;
  p.n_rows = N;
  p.tile_keys = tile_keys;
  p.n_stages = n_stages;
  p.off_mrg = off_mrg;
  p.off_small = off_small;
  p.idesc_qk = make_idesc(128, N, false, false);
  p.idesc_pv = make_idesc(kD, N, true, true);
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
  p.prefetch_next = prefetch_next ? 1 : 0;
  p.stall_first = (a.flags & FALCON_ATTN_TEST_STALL) ? 1 : 0;
  if (a.tree.prefix_len_host && a.tree.node_off_host && B <= kHostSeqs) {
    p.have_host = 1;
    for (int i = 0; i <= B; ++i) p.h_node_off[i] = a.tree.node_off_host[i];
    for (int i = 0; i < B; ++i) p.h_prefix[i] = a.tree.prefix_len_host[i];
    for (int i = 0; i < B; ++i) p.h_order[i] = i;
    std::stable_sort(p.h_order, p.h_order + B, [&](int x, int y) {
      return p.h_prefix[x] + (p.h_node_off[x + 1] - p.h_node_off[x]) > p.h_prefix[y] + (p.h_node_off[y + 1] - p.h_node_off[y]);
    });
  }

  FALCON_TRACE_LAUNCH(p)

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(splits, Hkv * n_units, B);
  cfg.blockDim = dim3(Var<kVar>::kThreads);
  cfg.dynamicSmemBytes = smem_bytes;
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
  cudaError_t e = (tile_keys == kBKMax && n_stages == 3)
                      ? cudaLaunchKernelEx(&cfg, tree_attn_tck_kernel<kVar, true>, mk, mv, mnk, mnv, p)
                      : cudaLaunchKernelEx(&cfg, tree_attn_tck_kernel<kVar, false>, mk, mv, mnk, mnv, p);
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

namespace {
// Nodes per unit: as many as the tree has, in steps that make the row count a multiple of 16, at most
// 128 rows.
int nodes_per_unit(const falcon_attn_args& a) {
  const int G = a.n_q_heads / a.n_kv_heads;
  const int gran = G >= 16 ? 1 : 16 / G;
  int q_nodes = 128 / G;
  const int want = (a.tree.max_tree + gran - 1) / gran * gran;
  return want < q_nodes ? want : q_nodes;
}
}  // namespace

// Where this kernel is the faster of the two tensor-core kernels (measured on the B200): blocks of
// at most 64 query rows (a 60-node tree with one query head per KV head), and launches with at least
// one unit per SM, which need no key splits.
bool tree_attn_tck_preferred(const falcon_ctx* ctx, const falcon_attn_args& a) {
  const int G = a.n_q_heads / a.n_kv_heads, q_nodes = nodes_per_unit(a);
  const int64_t units = static_cast<int64_t>(a.n_kv_heads) * ((a.tree.max_tree + q_nodes - 1) / q_nodes) * a.tree.batch;
  return q_nodes * G <= 64 || units >= ctx->sm_count;
}

int launch_tree_attn_tck(falcon_ctx* ctx, const falcon_attn_args& a, cudaStream_t s) {
  const int G = a.n_q_heads / a.n_kv_heads, q_nodes = nodes_per_unit(a);
  const int rows = q_nodes * G;
  if (rows <= 64) return launch_impl<0>(ctx, a, s, q_nodes);
  if (rows <= 80) return launch_impl<1>(ctx, a, s, q_nodes);
  return launch_impl<2>(ctx, a, s, q_nodes);
}

}  // namespace falcon
