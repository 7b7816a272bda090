// falcon_tree_attn, tensor-core kernel for sm_100a (head_dim 128, tree K/V in the cache).
//
// Work decomposition: one thread-block cluster per (sequence, KV head, tile of 128
// query rows); query row m of a KV head is (tree node m / G, query head m % G), so
// grouped-query heads share the K/V stream.  The cluster's CTAs split the key range
// (prefix + tree) into contiguous runs of 64-key tiles; each CTA runs a flash-style
// loop over its run, then pushes its partial (max, sum, O) rows into the shared
// memory of the CTA that owns them (distributed shared memory), one cluster barrier,
// and every CTA normalises and stores its share of the rows.  No partial result
// touches global memory.
//
// Inside a CTA (320 threads):
//   warp 0    TMA producer: the Q tile first, then K and V tiles (bf16, 128-byte swizzle) into a
//             4-stage ring, completion on mbarriers; the first loads are issued by several warps.
//   warp 1    one elected lane issues tcgen05.mma (the whole warp runs the loop).
//             S = Q.K^T (M=128, N=64, K=128) reads Q and the K tile from shared memory;
//             O += P.V (M=128, N=128, K=64) reads P from TMEM and the V tile from shared memory.
//             tcgen05.commit signals the consumers.
//   warps 2-9 softmax, one thread per (query row, stream or copy): per tile tcgen05.ld of the
//             score row, tree mask from the node's ancestor bit set, online softmax with a lazily
//             updated maximum (the accumulator is rescaled only when a weight would exceed 2^8),
//             P written back to TMEM as packed bf16.  Units of more than 64 rows run two streams
//             (warps 2-5 the even tiles, 6-9 the odd ones, one accumulator each, folded at the
//             end); units of at most 64 rows hold the rows twice (lanes 0-63 and 64-127) and give
//             each copy half of every tile's key columns (warps 2-5 only).
// The partial rows cross the cluster as bf16 columns plus fp32 (max, sum).  All three falcon
// kernels are launched programmatically dependent: set-up that touches no global memory runs
// before griddepcontrol.wait and overlaps the previous kernel's drain.
// Every mbarrier wait is bounded; a wait that runs out sets FALCON_DEV_TIMEOUT in the
// status word, and the CTA still reaches the cluster barrier and frees its TMEM.
#include <cuda.h>

#include <mutex>

#include "tc_util.cuh"

// Profiling hook, off by default: a build may predefine it to record per-phase time stamps.
#ifndef FALCON_TRACE
#define FALCON_TRACE(who, id)
#define FALCON_TRACE_PARAMS
#define FALCON_TRACE_LAUNCH(p)
#endif

namespace falcon {
namespace {

constexpr int kD = 128;
constexpr int kBM = 128;          // query rows per CTA (TMEM lanes)
constexpr int kBN = 64;           // keys per tile
constexpr int kStages = 4;         // ring depth: what shared memory leaves room for next to Q and the merge area
// Tiles requested ahead of the consumer.  Small on purpose: everything a CTA asks for at once
// arrives together (the memory system serves the whole GPU's requests fairly), so a deep burst only
// delays the first tile; the ring still lets the producer run ahead once tiles are consumed.
constexpr int kPrefetch = 2;
// Warp roles.  A CTA's warps start one after the other (the tenth about 800 cycles after the first),
// so the two warps with the longest set-up come first: 0 producer, 1 MMA, 2-9 softmax (TMEM
// quadrant = warp % 4, stream = (warp - 2) / 4).
constexpr int kTcThreads = 320;
constexpr int kWarpProducer = 0;
constexpr int kWarpMma = 1;
constexpr int kWarpSm0 = 2;
constexpr int kMaxSplits = 8;
constexpr int kHostSeqs = 8;
constexpr float kRescaleLimit = 256.f;  // largest weight tolerated before the row maximum is refreshed

constexpr uint32_t kTileBytes = kBN * kD * 2;      // 16 KB: two 64-column halves of 8 KB
constexpr uint32_t kHalfTile = kBN * 128;          // 8 KB
constexpr uint32_t kQBytes = kBM * kD * 2;          // 32 KB: two 64-column halves of 16 KB
constexpr uint32_t kOffQ = 0;
constexpr uint32_t kOffKV = kOffQ + kQBytes;
constexpr uint32_t kKVBytes = kStages * 2 * kTileBytes;  // 128 KB
// Merge: a CTA that has finished its key range stages its partial rows over its own (now idle) Q
// tile and K/V ring and bulk-copies each owner's rows into that owner's merge area, which is
// dedicated memory: a peer may still be in its main loop when the rows arrive.  A row is the 128
// accumulator columns rounded to bf16 (the transfer between CTAs is what bounds the merge, and the
// output is bf16 anyway), then the row's running maximum and sum in fp32, padded to kMrgRowBytes.
constexpr int kMrgRows = kBM + kMaxSplits;          // rows_per * n_splits <= n_valid + n_splits - 1
constexpr uint32_t kMrgRowBytes = kD * 2 + 16;      // 272-byte rows: 16-byte accesses of 32 lanes hit all banks evenly
constexpr uint32_t kOffStage = 0;                   // [row][kMrgRowBytes] staging of this CTA's partial rows
constexpr uint32_t kOffMrg = kOffKV + kKVBytes;
constexpr uint32_t kMrgBytes = kMrgRows * kMrgRowBytes;
constexpr uint32_t kSmemBytes = kOffMrg + kMrgBytes;
constexpr uint32_t kSmemAlloc = kSmemBytes + 1024;  // room to align the base to 1 KB
static_assert(kBM * kMrgRowBytes <= kOffMrg, "staging must fit over Q and the K/V ring");

// tensor memory columns (32-bit each, 128 lanes)
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemO = 0;      // 2 x 128 columns: fp32 accumulators (one per softmax stream)
constexpr uint32_t kTmemS = 256;    // 2 x 64 columns: fp32 scores
constexpr uint32_t kTmemP = 384;    // 2 x 32 columns: bf16 pairs

enum {
  kBarQ = 0,                         // the Q tile has landed in shared memory
  kBarKVFull = 1,                    // [kStages] K and V tile of the stage have landed
  kBarKVEmpty = kBarKVFull + kStages, // [kStages]
  kBarSFull = kBarKVEmpty + kStages, // [2]
  kBarPFull = kBarSFull + 2,         // [2]
  kBarPEmpty = kBarPFull + 2,        // [2]  also "P.V of tile j finished"
  kBarODone = kBarPEmpty + 2,
  kBarMrg = kBarODone + 1,           // all partial rows this CTA owns have arrived
  kNumBars = kBarMrg + 1
};

struct TcParams {
  int32_t Hq, Hkv, G, s_cap, total_nodes;
  uint32_t q_half_bytes;  // distance between the two 64-column halves of the Q tile in shared memory
  uint32_t q_box_bytes;   // bytes one Q load brings in
  float scale_log2;
  const int32_t* node_off;
  const int32_t* parent;
  const int32_t* prefix_len;
  int32_t* status;
  const uint64_t* tree_mask;
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  // Per-sequence scalars from the caller's host copies (batches of up to kHostSeqs sequences):
  // with them the first loads do not have to wait for a round trip to global memory.
  int32_t have_host;
  int32_t early_prefix;  // prefix tiles may be requested before the previous kernel has completed
  int32_t stall_first;   // test hook: tile 0 is never requested (a bounded wait then runs out)
  int32_t h_node_off[kHostSeqs + 1];
  int32_t h_prefix[kHostSeqs];
  FALCON_TRACE_PARAMS
};

using namespace tc;

// instruction descriptors: A K-major; B K-major (K tile) or MN-major (V tile)
constexpr uint32_t kIdescQK = make_idesc(kBM, kBN, false, false);
constexpr uint32_t kIdescPV = make_idesc(kBM, kD, false, true);


// ------------------------------------------------------------------------------------ kernel
// kDup: the tile has at most 64 query rows.  They are then held twice, in TMEM lanes 0-63 and 64-127
// (the Q tile is loaded twice), and the two copies share every key tile: lanes 0-63 take its key
// columns 0-31, lanes 64-127 columns 32-63, each with its own running maximum and sum, as if they
// were two more key splits.  All four SM sub-partitions then work on the exponentials, which is
// what bounds a tile, instead of two.
template <bool kDup>
__global__ void __launch_bounds__(kTcThreads, 1)
tree_attn_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const TcParams p) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t s_bars[kNumBars];
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;
  __shared__ float2 s_ml[2][kBM];  // [stream][row]: running maximum and sum, exchanged once after the loop

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  FALCON_TRACE(tid == 0, 0);
  const int n_splits = gridDim.x, split = blockIdx.x;  // cluster = all CTAs of a row of the grid
  const int kvh = blockIdx.y % p.Hkv, mtile = blockIdx.y / p.Hkv, b = blockIdx.z;
  const int G = p.G;

  // What touches no global memory comes first: tensor-map prefetch, barrier initialisation (all but
  // the two whose count depends on the tree), tensor memory.  Under programmatic dependent launch
  // this part runs while the previous kernel of the stream is still finishing.
  const uint32_t bars = smem_u32(s_bars);
  auto bar = [&](int i) { return bars + 8u * static_cast<uint32_t>(i); };
  if (warp == kWarpProducer) {
    if (lane == 0) {
      s_abort = 0;
      prefetch_tmap(&tm_q);
      prefetch_tmap(&tm_k);
      prefetch_tmap(&tm_v);
    }
    if (lane < kNumBars && lane != kBarPFull && lane != kBarPFull + 1) mbar_init(bar(lane), 1);  // barrier i: lane i
  } else if (warp == kWarpMma) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  int node_base = 0, T_real = 0, L_raw = 0;
  int n_early = 0;  // K/V tiles requested before the wait below
  if (p.have_host) {
    node_base = p.h_node_off[b];
    T_real = p.h_node_off[b + 1] - node_base;
    L_raw = p.h_prefix[b];
    // Prefix rows that the caller declares stable (written before the kernel that precedes this one
    // in the stream started) may be requested while that kernel is still finishing.
    if (p.early_prefix && warp == kWarpProducer) {
      __syncwarp();
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      if (lane == 0 && mtile * kBM < min(T_real, FALCON_T_MAX) * G) {
        const int Tq = min(T_real, FALCON_T_MAX), Lq = min(max(L_raw, 0), p.s_cap);
        const int Sv = min(max(L_raw, 0) + Tq, p.s_cap);
        const int nt = (Sv + kBN - 1) / kBN;
        const int kb = min(Sv, ((split * nt + n_splits - 1) / n_splits) * kBN);
        const int ke = min(Sv, (((split + 1) * nt + n_splits - 1) / n_splits) * kBN);
        const int nm = (ke - kb + kBN - 1) / kBN;
        for (int j = 0; j < min(nm, kPrefetch) && kb + (j + 1) * kBN <= Lq; ++j) {
          ++n_early;
          if (j == 0 && p.stall_first) continue;
          const uint32_t kdst = smem_base + kOffKV + j * 2 * kTileBytes;
          mbar_expect_tx(bar(kBarKVFull + j), 2 * kTileBytes);
          load_kv_tile(kdst, &tm_k, bar(kBarKVFull + j), kb + j * kBN, kvh, b);
          load_kv_tile(kdst + kTileBytes, &tm_v, bar(kBarKVFull + j), kb + j * kBN, kvh, b);
        }
      }
    }
  }
  // Everything below may read what earlier kernels of the stream wrote (tree arrays, q, the tree's
  // K/V rows) and writes `out`: wait until they have completed.  Then let the next kernel's CTAs
  // be scheduled as this grid's CTAs leave their SMs (a no-op without programmatic launch).
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (!p.have_host) {
    node_base = p.node_off[b];
    T_real = p.node_off[b + 1] - node_base;
    L_raw = p.prefix_len[b];
  }
  const int T = min(T_real, FALCON_T_MAX);
  const int rows_total = T * G;
  if (mtile * kBM >= rows_total) {  // no query rows here; same decision in every CTA of the cluster
    tc_fence_before();
    __syncthreads();
    if (warp == kWarpMma) {
      tc_fence_after();
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(s_tmem_base), "r"(kTmemCols) : "memory");
    }
    return;
  }
  const int n_valid = min(kBM, rows_total - mtile * kBM);
  const int L = max(L_raw, 0);
  const int Lc = min(L, p.s_cap);
  const int S_valid = min(L + T, p.s_cap);  // keys that exist below the cache capacity
  // Whole tiles per split, as even as they go (an iteration costs about the same whatever part of
  // its 64 keys is real, so fewer iterations beat equal key counts).  The boundaries are rounded
  // up, so a longer run goes to an early split: the last one has the tree's tiles, whose masked
  // softmax pass is the slowest, and should not be the cluster's straggler as well.
  const int n_tiles = (S_valid + kBN - 1) / kBN;
  const int key_begin = min(S_valid, ((split * n_tiles + n_splits - 1) / n_splits) * kBN);
  const int key_end = min(S_valid, (((split + 1) * n_tiles + n_splits - 1) / n_splits) * kBN);
  const int n_my = (key_end - key_begin + kBN - 1) / kBN;

  unsigned char* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  volatile int* abort_flag = &s_abort;

  // merge geometry: CTA `rank` owns rows [rank * rows_per, ...) of the tile
  const int rows_per = (n_valid + n_splits - 1) / n_splits;

  constexpr int kCols = kDup ? 32 : 64;  // key columns of a tile that one softmax thread handles
  constexpr int kGroups = kDup ? 2 : 1;  // partial results per row and CTA
  // Softmax streams: with two, warps 2-5 take the even tiles of the CTA's run and warps 6-9 the odd
  // ones, each stream with its own maximum, sum and accumulator.  Warps w and w+4 sit on the same
  // scheduler and reach the same TMEM lanes, so one stream's exponentials fill the gaps of the
  // other's loads, stores and barrier traffic, and after the loop the two threads of a row fold
  // the two accumulators into one partial result at no extra traffic.
  constexpr int kStreams = kDup ? 1 : 2;
  const int n_vs = kGroups * n_splits;   // partial results per row in the whole cluster
  const bool merge = kDup || n_splits > 1;
  const int row_warps = (n_valid + 31) >> 5;
  const int n_sm_warps = kGroups * row_warps;  // softmax warps that own at least one query row
  const int q4 = warp & 3;
  const int lane_row = q4 * 32 + lane;                       // TMEM lane, and the staging slot of its partial row
  const int grp = kDup ? (q4 >> 1) : 0;                      // which half of a tile's key columns
  const int row = kDup ? (q4 & 1) * 32 + lane : lane_row;    // query row of the tile
  const bool is_sm = warp >= kWarpSm0 && warp < kWarpSm0 + 4 * kStreams;
  const int strm = kStreams == 2 ? (((warp - kWarpSm0) >> 2) & 1) : 0;
  const bool valid = is_sm && row < n_valid;
  const bool warp_valid = is_sm && (row - lane) < n_valid;

  if (warp == kWarpProducer) {
    FALCON_TRACE(lane == 0, 1);
    if (lane == kBarPFull || lane == kBarPFull + 1) mbar_init(bar(lane), n_sm_warps);  // one arrival per softmax warp
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncwarp();
    // First loads, by this warp alone and before the CTA-wide barrier below (the CTA's last warps
    // start hundreds of cycles after this one): the barriers they land on were initialised by this
    // warp's own lanes.  Q goes first so that it is not queued behind K/V.
    if (lane == 0) {
      if (n_splits > 1) {
        // this CTA will receive rows_mine rows of every other CTA's partial results
        const int r0 = split * rows_per;
        const int mine = max(0, min(n_valid, r0 + rows_per) - r0);
        mbar_expect_tx(bar(kBarMrg), static_cast<uint32_t>((n_vs - kGroups) * mine) * kMrgRowBytes);
      }
      if (n_my > 0) {
        const int node0 = node_base + mtile * (kBM / G);
        if (kDup) {  // one load per 64-column half and copy (the second copy 64 rows further down)
          mbar_expect_tx(bar(kBarQ), 4 * p.q_box_bytes);
#pragma unroll
          for (int c = 0; c < 2; ++c)
#pragma unroll
            for (int h = 0; h < 2; ++h)
              tma_load_5d(smem_base + kOffQ + h * p.q_half_bytes + c * 64 * 128, &tm_q, bar(kBarQ), 0, 0, kvh, node0, h);
        } else {
          mbar_expect_tx(bar(kBarQ), p.q_box_bytes);
          tma_load_5d(smem_base + kOffQ, &tm_q, bar(kBarQ), 0, 0, kvh, node0, 0);
        }
      }
      const int pre = min(n_my, kPrefetch);
      for (int j = n_early; j < pre; ++j) {
        if (j == 0 && p.stall_first) continue;
        const uint32_t kdst = smem_base + kOffKV + j * 2 * kTileBytes;
        mbar_expect_tx(bar(kBarKVFull + j), 2 * kTileBytes);
        load_kv_tile(kdst, &tm_k, bar(kBarKVFull + j), key_begin + j * kBN, kvh, b);
        load_kv_tile(kdst + kTileBytes, &tm_v, bar(kBarKVFull + j), key_begin + j * kBN, kvh, b);
      }
      if (split == 0 && mtile == 0 && kvh == 0 && (L + T > p.s_cap || T_real > FALCON_T_MAX))
        dev_status_or(p.status, b, FALCON_DEV_CAPACITY);
      FALCON_TRACE(true, 2);
    }
    __syncwarp();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = s_tmem_base;
  FALCON_TRACE(tid == 0, 4);
  // Cluster phase 1: "my merge barrier exists".  Arrive now, wait just before the first remote copy.
  if (merge) cluster_arrive();

  if (warp == kWarpProducer) {
    // ================================ TMA producer (ring refills) ================================
    if (lane == 0) {
      int issued = min(n_my, kPrefetch);
      for (int j = kPrefetch; j < n_my; ++j) {
        const int st = j % kStages, u = j / kStages;
        // Ramp: the stages not used yet are filled one by one as earlier tiles land (a deep first
        // burst would only delay the first tile); after that a tile is requested as soon as its
        // stage has been consumed, which keeps the whole ring in flight.
        if (u == 0) {
          const int jl = j - kPrefetch;
          if (!mbar_wait(bar(kBarKVFull + jl % kStages), (jl / kStages) & 1, abort_flag)) break;
        } else if (!mbar_wait(bar(kBarKVEmpty + st), (u - 1) & 1, abort_flag)) {
          break;
        }
        const int k0 = key_begin + j * kBN;
        const uint32_t kdst = smem_base + kOffKV + st * 2 * kTileBytes;
        const uint32_t vdst = kdst + kTileBytes;
        mbar_expect_tx(bar(kBarKVFull + st), 2 * kTileBytes);
        load_kv_tile(kdst, &tm_k, bar(kBarKVFull + st), k0, kvh, b);
        load_kv_tile(vdst, &tm_v, bar(kBarKVFull + st), k0, kvh, b);
        issued = j + 1;
      }
      if (*abort_flag) {
        // Some wait gave up.  What was asked for still arrives: stay until it has (bounded, without
        // looking at the abort flag), so that no copy is in flight into this CTA's shared memory
        // when it leaves.
        auto drain = [&](uint32_t b_, uint32_t parity) {
          for (uint32_t it = 0; it < (1u << 20); ++it) {
            uint32_t ok;
            asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                         : "=r"(ok)
                         : "r"(b_), "r"(parity)
                         : "memory");
            if (ok) return;
          }
        };
        if (n_my > 0) drain(bar(kBarQ), 0);
        for (int j = max(0, issued - kStages); j < issued; ++j)
          if (!(j == 0 && p.stall_first)) drain(bar(kBarKVFull + j % kStages), (j / kStages) & 1);
      }
    }
  } else if (warp == kWarpMma) {
    // ================================ MMA issuer ================================
    // The whole warp runs this loop (descriptors stay in uniform registers, which keeps the
    // issue cost per tcgen05.mma low); one elected lane issues.
    if (n_my > 0) {
      uint32_t elected;
      asm volatile("{ .reg .pred p; elect.sync _|p, 0xffffffff; selp.u32 %0, 1, 0, p; }" : "=r"(elected));
      bool ok = mbar_wait_warp(bar(kBarQ), 0, abort_flag);
      FALCON_TRACE(elected, 5);
      auto issue_qk = [&](int j) -> bool {
        const int st = j % kStages, sb = j & 1;
        if (!mbar_wait_warp(bar(kBarKVFull + st), (j / kStages) & 1, abort_flag)) return false;
        FALCON_TRACE(elected && j < 6, 10 + 4 * j);
        tc_fence_after();
        const uint32_t kbase = smem_base + kOffKV + st * 2 * kTileBytes;
        if (elected) {
#pragma unroll
          for (int kk = 0; kk < kD / 16; ++kk) {
            // Q and K tiles: K-major, 16 head-dim columns = 32 bytes inside the 128-byte swizzle row
            const uint64_t ad = smem_desc(smem_base + kOffQ + (kk >> 2) * p.q_half_bytes + (kk & 3) * 32, 16, 1024);
            const uint64_t bd = smem_desc(kbase + (kk >> 2) * kHalfTile + (kk & 3) * 32, 16, 1024);
            umma_bf16_ss(tmem_base + kTmemS + sb * kBN, ad, bd, kIdescQK, kk > 0 ? 1u : 0u);
          }
          umma_commit(bar(kBarSFull + sb));
          FALCON_TRACE(j < 6, 11 + 4 * j);
        }
        __syncwarp();
        return true;
      };
      auto issue_pv = [&](int t) {
        const int st = t % kStages, pb = t & 1;
        const uint32_t vbase = smem_base + kOffKV + st * 2 * kTileBytes + kTileBytes;
        const uint32_t acc = tmem_base + kTmemO + (kStreams == 2 ? pb * kD : 0);
        if (elected) {
#pragma unroll
          for (int kk = 0; kk < kBN / 16; ++kk) {
            // P: 16 keys = 8 packed columns; V: MN-major, 16 keys = 2 KB, the two 64-column halves 8 KB apart
            const uint64_t bd = smem_desc(vbase + kk * 2048, kHalfTile, 1024);
            umma_bf16_ts(acc, tmem_base + kTmemP + pb * 32 + kk * 8, bd, kIdescPV, (t >= kStreams || kk > 0) ? 1u : 0u);
          }
          umma_commit(bar(kBarKVEmpty + st));
          umma_commit(bar(kBarPEmpty + pb));
          FALCON_TRACE(t < 6, 13 + 4 * t);
        }
        __syncwarp();
      };
      // Two tiles of scores are always in flight (one per S buffer).  When P(t) is there, S buffer
      // t & 1 has been read, so Q.K^T of tile t+2 can go into it.  It is issued after P.V of tile t:
      // the commit behind S(t+2) then also covers that P.V, which is what tells the softmax warps
      // that P buffer t & 1 may be overwritten.
      ok = ok && issue_qk(0);
      if (ok && n_my > 1) ok = issue_qk(1);
      for (int t = 0; ok && t < n_my; ++t) {
        const int pb = t & 1;
        FALCON_TRACE(elected && t < 6, 113 + (t - 0));
        if (!mbar_wait_warp(bar(kBarPFull + pb), (t >> 1) & 1, abort_flag)) { ok = false; break; }
        FALCON_TRACE(elected && t < 6, 12 + 4 * t);
        tc_fence_after();
        issue_pv(t);
        if (t + 2 < n_my) ok = issue_qk(t + 2);
      }
      if (elected) umma_commit(bar(kBarODone));  // fires once every MMA issued so far has finished
      __syncwarp();
    }
  } else if (warp_valid) {
    // ================================ softmax / correction (warps that own query rows) ================================
    const uint32_t tmem_lane = tmem_base + (static_cast<uint32_t>(q4 * 32) << 16);
    const int sm_idx = (grp * row_warps + (row >> 5)) * 32 + lane;  // index among the CTA's working softmax threads

    uint64_t anc_lo = 0, anc_hi = 0;
    if (valid) {
      const int node = (mtile * kBM + row) / G;
      bool bad = false;
      if (p.tree_mask) {
        anc_lo = p.tree_mask[2 * static_cast<int64_t>(node_base + node)];
        anc_hi = p.tree_mask[2 * static_cast<int64_t>(node_base + node) + 1];
      } else {
        bad = !ancestor_mask(p.parent + node_base, T, node, anc_lo, anc_hi);
        if (node == 0 && p.parent[node_base] != -1) bad = true;
      }
      if (bad && split == 0 && kvh == 0) dev_status_or(p.status, b, FALCON_DEV_BAD_TREE);
      const int nt = S_valid - Lc;  // tree keys that can be read (<= T)
      if (nt < 64) {
        anc_hi = 0;
        anc_lo &= (nt <= 0) ? 0ull : ((1ull << nt) - 1ull);
      } else if (nt < 128) {
        anc_hi &= (nt == 64) ? 0ull : ((1ull << (nt - 64)) - 1ull);
      }
    }
    if constexpr (kDup) {  // the key columns of the other group stay zero in this group's rows of both P buffers
      uint32_t z[16];
#pragma unroll
      for (int c = 0; c < 16; ++c) z[c] = 0u;
      FALCON_TMEM_ST16(tmem_lane + kTmemP + (grp ^ 1) * 16, z);
      FALCON_TMEM_ST16(tmem_lane + kTmemP + 32 + (grp ^ 1) * 16, z);
      tmem_wait_st();
    }
    float m_used = -INFINITY, l_sum = 0.f;
    const float scale = p.scale_log2;

    const uint32_t tmem_acc = tmem_lane + kTmemO + strm * kD;  // this stream's accumulator
    for (int j = strm; j < n_my; j += kStreams) {
      const int sb = j & 1, u2 = j >> 1, st = j % kStages;
      const int k0 = key_begin + j * kBN;
      if (!mbar_wait_warp(bar(kBarSFull + sb), u2 & 1, abort_flag)) break;
      FALCON_TRACE(tid == 0 && j < 6, 40 + 4 * j);
      tc_fence_after();
      uint32_t sr[kCols];
      FALCON_TMEM_LD32(tmem_lane + kTmemS + sb * kBN + grp * 32, sr);
      if constexpr (!kDup) FALCON_TMEM_LD32(tmem_lane + kTmemS + sb * kBN + 32, (sr + 32));
      tmem_wait_ld();
      FALCON_TRACE(tid == 0 && j < 6, 41 + 4 * j);

      // the sequence's last tile: rows of V past the last key may hold anything (0 x NaN = NaN in the MMA)
      if (k0 + kBN > S_valid) {
        if (!mbar_wait_warp(bar(kBarKVFull + st), (j / kStages) & 1, abort_flag)) break;
        const int nv = S_valid - k0;  // 1..63 rows are real
        unsigned char* vtile = smem_gen + kOffKV + st * 2 * kTileBytes + kTileBytes;
        const int chunks = (kBN - nv) * 8;
        for (int c = sm_idx; c < 2 * chunks; c += 32 * n_sm_warps) {
          const int half = c / chunks, cc = c % chunks;
          *reinterpret_cast<uint4*>(vtile + half * kHalfTile + nv * 128 + cc * 16) = make_uint4(0, 0, 0, 0);
        }
        fence_async_smem();
      }

      uint32_t pk[kCols / 2];
      float alpha = 1.f;
      bool need_rescale = false;
      if (valid) {
        // scores stay raw; exp2(s * scale - m) is one FFMA + one MUFU per element (scale > 0 is
        // guaranteed by the launcher, so a maximum can be taken on the raw scores)
        float s[kCols];
        if (k0 + kBN <= min(Lc, key_end)) {
#pragma unroll
          for (int c = 0; c < kCols; ++c) s[c] = __uint_as_float(sr[c]);
        } else {
          uint64_t vis = window64(anc_lo, anc_hi, k0 - Lc);
          if (key_end - k0 < kBN) vis &= (1ull << (key_end - k0)) - 1ull;  // keys of the next split
          const uint32_t vlo = static_cast<uint32_t>(vis), vhi = static_cast<uint32_t>(vis >> 32);
#pragma unroll
          for (int c = 0; c < kCols; ++c) {
            const uint32_t w = kDup ? (grp ? vhi : vlo) : (c < 32 ? vlo : vhi);
            s[c] = ((w >> (c & 31)) & 1u) ? __uint_as_float(sr[c]) : -INFINITY;
          }
        }
        // One pass of exponentials against the maximum known so far.  The largest p tells whether
        // that maximum is still good enough (p <= 2^8); only the first tile of a row, or a row whose
        // scores jumped, needs the true maximum of this tile first.
        float pmx0 = 0.f, pmx1 = 0.f, add0 = 0.f, add1 = 0.f, add2 = 0.f, add3 = 0.f;
        auto exp_pass = [&](float neg_m) {
          pmx0 = pmx1 = add0 = add1 = add2 = add3 = 0.f;
#pragma unroll
          for (int c = 0; c < kCols / 2; c += 2) {
            const float p0 = ex2(fmaf(s[2 * c], scale, neg_m)), p1 = ex2(fmaf(s[2 * c + 1], scale, neg_m));
            const float p2 = ex2(fmaf(s[2 * c + 2], scale, neg_m)), p3 = ex2(fmaf(s[2 * c + 3], scale, neg_m));
            add0 += p0;
            add1 += p1;
            add2 += p2;
            add3 += p3;
            pmx0 = fmaxf(pmx0, fmaxf(p0, p1));
            pmx1 = fmaxf(pmx1, fmaxf(p2, p3));
            const __nv_bfloat162 h0 = __floats2bfloat162_rn(p0, p1), h1 = __floats2bfloat162_rn(p2, p3);
            pk[c] = *reinterpret_cast<const uint32_t*>(&h0);
            pk[c + 1] = *reinterpret_cast<const uint32_t*>(&h1);
          }
        };
        bool redo = (m_used == -INFINITY);
        if (!redo) {
          exp_pass(-m_used);
          redo = !(fmaxf(pmx0, pmx1) <= kRescaleLimit);  // also catches an overflow to +inf
        }
        if (redo) {
          float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
          for (int c = 0; c < kCols; c += 4) {
            mx0 = fmaxf(mx0, s[c]);
            mx1 = fmaxf(mx1, s[c + 1]);
            mx2 = fmaxf(mx2, s[c + 2]);
            mx3 = fmaxf(mx3, s[c + 3]);
          }
          const float tmax = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * scale;  // -inf stays -inf
          if (m_used != -INFINITY) {  // what is accumulated so far moves to the new maximum
            alpha = ex2(m_used - tmax);
            l_sum *= alpha;
            need_rescale = true;
          }
          m_used = tmax;
          exp_pass(m_used == -INFINITY ? 0.f : -m_used);
        }
        FALCON_TRACE(tid == 0 && j < 6 && pmx0 >= 0.f, 83 + 4 * j);
        l_sum += (add0 + add1) + (add2 + add3);
      } else {
#pragma unroll
        for (int c = 0; c < kCols / 2; ++c) pk[c] = 0u;
      }

      FALCON_TRACE(tid == 0 && j < 6 && l_sum >= 0.f, 42 + 4 * j);
      // P buffer sb is free: the commit behind S(j) covers every MMA issued before it, and P.V of
      // tile j-2 was issued before Q.K^T of tile j.

      // rare: the row maximum jumped; rescale the accumulator before this tile is added (the
      // stream's previous tile must have been added first)
      if (__any_sync(0xffffffffu, need_rescale) && j >= kStreams) {
        const int jp = j - kStreams;
        if (!mbar_wait_warp(bar(kBarPEmpty + (jp & 1)), (jp >> 1) & 1, abort_flag)) break;
        tc_fence_after();
#pragma unroll 1
        for (int ch = 0; ch < 4; ++ch) {
          uint32_t o[32];
          FALCON_TMEM_LD32(tmem_acc + ch * 32, o);
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
          FALCON_TMEM_ST32(tmem_acc + ch * 32, o);
        }
      }

      if constexpr (kDup) {
        FALCON_TMEM_ST16(tmem_lane + kTmemP + sb * 32 + grp * 16, pk);
      } else {
        FALCON_TMEM_ST32(tmem_lane + kTmemP + sb * 32, pk);
      }
      FALCON_TRACE(tid == 0 && j < 6, 81 + 4 * j);
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(kBarPFull + sb));
      FALCON_TRACE(tid == 0 && j < 6, 43 + 4 * j);
      FALCON_TRACE(tid == 128 && j < 6, 107 + (j - 0));
    }

    // ---- this split's partial rows: straight to global (one partial per row) or staged for the merge ----
    bool have = (n_my > 0) && !*abort_flag;
    if (have) have = mbar_wait_warp(bar(kBarODone), 0, abort_flag);
    FALCON_TRACE(tid == 0, 70);
    tc_fence_after();
    const bool write = have && valid;
    if constexpr (kStreams == 2) {
      // Fold the two streams' accumulators: the two threads of a row (same lanes, so each reaches
      // both accumulators) swap their maximum and sum, then each takes 64 of the 128 columns.
      s_ml[strm][row] = make_float2(m_used, l_sum);
      asm volatile("bar.sync %0, 64;" ::"r"(1 + q4) : "memory");
      const float2 ot = s_ml[strm ^ 1][row];
      const float gm = fmaxf(m_used, ot.x);
      const float w_me = (m_used == -INFINITY) ? 0.f : ex2(m_used - gm);
      const float w_ot = (ot.x == -INFINITY) ? 0.f : ex2(ot.x - gm);
      const float l_row = l_sum * w_me + ot.y * w_ot;
      const float inv = merge ? 1.f : (l_row > 0.f ? 1.f / l_row : 0.f);
      // weights of accumulators 0 and 1, normalisation folded in
      const float f0 = (strm == 0 ? w_me : w_ot) * inv, f1 = (strm == 0 ? w_ot : w_me) * inv;
      // Accumulator 1 holds anything when the CTA's run is a single tile; otherwise both are finite
      // (a row whose keys were all masked in a stream has weight 0 and an all-zero accumulator).
      const bool two = n_my > 1;
      const int mg = mtile * kBM + row;
      __nv_bfloat16* dst =
          p.out + (static_cast<int64_t>(node_base + mg / G) * p.Hq + kvh * G + mg % G) * kD + strm * 64;
      unsigned char* stage = smem_gen + kOffStage + lane_row * kMrgRowBytes + strm * 128;
      if (have) {
#pragma unroll 1
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t o0[32], o1[32];
          FALCON_TMEM_LD32(tmem_lane + kTmemO + strm * 64 + ch * 32, o0);
          if (two) FALCON_TMEM_LD32(tmem_lane + kTmemO + kD + strm * 64 + ch * 32, o1);
          tmem_wait_ld();
          if (valid) {
            uint32_t h[16];
            if (two) {
#pragma unroll
              for (int c = 0; c < 16; ++c) {
                const float a = fmaf(__uint_as_float(o1[2 * c]), f1, __uint_as_float(o0[2 * c]) * f0);
                const float bq = fmaf(__uint_as_float(o1[2 * c + 1]), f1, __uint_as_float(o0[2 * c + 1]) * f0);
                const __nv_bfloat162 hh = __floats2bfloat162_rn(a, bq);
                h[c] = *reinterpret_cast<const uint32_t*>(&hh);
              }
            } else {
#pragma unroll
              for (int c = 0; c < 16; ++c) {
                const __nv_bfloat162 hh =
                    __floats2bfloat162_rn(__uint_as_float(o0[2 * c]) * f0, __uint_as_float(o0[2 * c + 1]) * f0);
                h[c] = *reinterpret_cast<const uint32_t*>(&hh);
              }
            }
            uint4* d4 = merge ? reinterpret_cast<uint4*>(stage + ch * 64) : reinterpret_cast<uint4*>(dst + ch * 32);
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) d4[c4] = make_uint4(h[4 * c4], h[4 * c4 + 1], h[4 * c4 + 2], h[4 * c4 + 3]);
          }
        }
      } else if (valid && !merge) {  // nothing was computed (a wait ran out): the row reads as zero
#pragma unroll
        for (int c4 = 0; c4 < 8; ++c4) reinterpret_cast<uint4*>(dst)[c4] = make_uint4(0u, 0u, 0u, 0u);
      }
      if (merge) {
        if (valid && strm == 0)
          *reinterpret_cast<float2*>(smem_gen + kOffStage + lane_row * kMrgRowBytes + kD * 2) =
              make_float2(write ? gm : -INFINITY, write ? l_row : 0.f);
        fence_async_smem();  // the bulk copies below read these rows through the async proxy
      }
    } else
    if (!merge) {
      const float inv = (write && l_sum > 0.f) ? 1.f / l_sum : 0.f;
      const int mg = mtile * kBM + row;
      __nv_bfloat16* dst = p.out + (static_cast<int64_t>(node_base + mg / G) * p.Hq + kvh * G + mg % G) * kD;
#pragma unroll 1
      for (int ch = 0; ch < 2; ++ch) {
        uint32_t o[64];
        FALCON_TMEM_LD32(tmem_lane + kTmemO + ch * 64, o);
        FALCON_TMEM_LD32(tmem_lane + kTmemO + ch * 64 + 32, (o + 32));
        tmem_wait_ld();
        if (valid) {
#pragma unroll
          for (int c8 = 0; c8 < 8; ++c8) {
            __align__(16) __nv_bfloat162 h[4];
#pragma unroll
            for (int c = 0; c < 4; ++c)
              h[c] = __floats2bfloat162_rn(__uint_as_float(o[8 * c8 + 2 * c]) * inv,
                                           __uint_as_float(o[8 * c8 + 2 * c + 1]) * inv);
            *reinterpret_cast<uint4*>(dst + ch * 64 + c8 * 8) = *reinterpret_cast<const uint4*>(h);
          }
        }
      }
    } else {
      // Q and the K/V ring are idle now (all of this CTA's MMAs have finished): stage lane -> [lane][kMrgRowBytes]
      unsigned char* stage = smem_gen + kOffStage + lane_row * kMrgRowBytes;
      if (have) {
#pragma unroll 1
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t o[64];
          FALCON_TMEM_LD32(tmem_lane + kTmemO + ch * 64, o);
          FALCON_TMEM_LD32(tmem_lane + kTmemO + ch * 64 + 32, (o + 32));
          tmem_wait_ld();
          if (valid) {
#pragma unroll
            for (int c8 = 0; c8 < 8; ++c8) {
              __align__(16) __nv_bfloat162 h[4];
#pragma unroll
              for (int c = 0; c < 4; ++c)
                h[c] = __floats2bfloat162_rn(__uint_as_float(o[8 * c8 + 2 * c]), __uint_as_float(o[8 * c8 + 2 * c + 1]));
              *reinterpret_cast<uint4*>(stage + ch * 128 + c8 * 16) = *reinterpret_cast<const uint4*>(h);
            }
          }
        }
      }
      if (valid)
        *reinterpret_cast<float2*>(stage + kD * 2) = make_float2(write ? m_used : -INFINITY, write ? l_sum : 0.f);
      fence_async_smem();  // the bulk copies below read these rows through the async proxy
    }
  }

  FALCON_TRACE(tid == 0, 71);
  // ================================ cluster merge ================================
  tc_fence_before();
  __syncthreads();
  FALCON_TRACE(tid == 0, 72);
  if (s_abort && tid == 0) dev_status_or(p.status, b, FALCON_DEV_TIMEOUT);
  if (merge) {
    cluster_wait();  // phase 1 (arrived long ago): every peer's merge barrier is initialised
    FALCON_TRACE(tid == 0, 73);
    if (warp == kWarpProducer && lane == 0) {
      // one bulk copy per other owner and partial result: the owner's rows are contiguous in the
      // staging area (this CTA's own rows are merged from there directly)
      for (int o = 0; o < n_splits; ++o) {
        const int r0 = o * rows_per;
        const int cnt = min(n_valid, r0 + rows_per) - r0;
        if (cnt <= 0) break;
        if (o == split) continue;
        const uint32_t peer_bar = map_to_rank(bar(kBarMrg), o);
#pragma unroll
        for (int g = 0; g < kGroups; ++g)
          bulk_copy_to_peer(
              map_to_rank(smem_base + kOffMrg + static_cast<uint32_t>((split * kGroups + g) * rows_per) * kMrgRowBytes, o),
              smem_base + kOffStage + static_cast<uint32_t>(g * 64 + r0) * kMrgRowBytes,
              static_cast<uint32_t>(cnt) * kMrgRowBytes, peer_bar);
      }
    }
    __syncwarp();
    const int row0 = split * rows_per;
    const int rows_mine = max(0, min(n_valid, row0 + rows_per) - row0);
    bool got = rows_mine == 0 || n_splits == 1 || mbar_wait_warp(bar(kBarMrg), 0, abort_flag);
    if (!got) {
      // This wait gave up (or another did).  Every peer still sends its rows, whatever happened to it,
      // so stay, without looking at the abort flag, until they have landed: the CTA must not reach the
      // exit barrier, and leave, while a copy into its merge area is in flight.  The rows stay unmerged.
      bool landed = false;
      for (uint32_t it = 0; it < (1u << 20) && !landed; ++it) {
        uint32_t ok;
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                     : "=r"(ok)
                     : "r"(bar(kBarMrg)), "r"(0u)
                     : "memory");
        landed = __all_sync(0xffffffffu, ok != 0);
      }
    }
    FALCON_TRACE(tid == 0, 74);
    const unsigned char* mrg = smem_gen + kOffMrg;
    const unsigned char* own = smem_gen + kOffStage + static_cast<uint32_t>(row0) * kMrgRowBytes;
    for (int item = tid; got && item < rows_mine * (kD / 8); item += kTcThreads) {
      const int rl = item / (kD / 8), c8 = item % (kD / 8);
      // all loads first (independent), then the arithmetic
      float2 m_l[kMaxSplits];
      uint4 x[kMaxSplits];  // 8 bf16 columns of each partial row
#pragma unroll
      for (int s = 0; s < kMaxSplits; ++s) {
        m_l[s] = make_float2(-INFINITY, 0.f);
        x[s] = make_uint4(0u, 0u, 0u, 0u);
        if (s < n_vs) {
          const unsigned char* rowp = (s / kGroups == split)
                                          ? own + static_cast<uint32_t>((s % kGroups) * 64 + rl) * kMrgRowBytes
                                          : mrg + static_cast<uint32_t>(s * rows_per + rl) * kMrgRowBytes;
          m_l[s] = *reinterpret_cast<const float2*>(rowp + kD * 2);
          x[s] = *reinterpret_cast<const uint4*>(rowp + c8 * 16);
        }
      }
      float gm = -INFINITY;
#pragma unroll
      for (int s = 0; s < kMaxSplits; ++s) gm = fmaxf(gm, m_l[s].x);
      float lsum = 0.f, acc[8];
#pragma unroll
      for (int c = 0; c < 8; ++c) acc[c] = 0.f;
#pragma unroll
      for (int s = 0; s < kMaxSplits; ++s) {
        if (m_l[s].x != -INFINITY) {  // a split that saw no key of this row has no valid columns
          const float w = ex2(m_l[s].x - gm);
          lsum = fmaf(m_l[s].y, w, lsum);
          const uint32_t xs[4] = {x[s].x, x[s].y, x[s].z, x[s].w};
#pragma unroll
          for (int c = 0; c < 4; ++c) {  // a bf16 is the upper half of the fp32 of the same value
            acc[2 * c] = fmaf(__uint_as_float(xs[c] << 16), w, acc[2 * c]);
            acc[2 * c + 1] = fmaf(__uint_as_float(xs[c] & 0xffff0000u), w, acc[2 * c + 1]);
          }
        }
      }
      const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
      const int mg = mtile * kBM + row0 + rl;
      __align__(16) __nv_bfloat162 h[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) h[c] = __floats2bfloat162_rn(acc[2 * c] * inv, acc[2 * c + 1] * inv);
      *reinterpret_cast<uint4*>(p.out + (static_cast<int64_t>(node_base + mg / G) * p.Hq + kvh * G + mg % G) * kD +
                                c8 * 8) = *reinterpret_cast<const uint4*>(h);
    }
    // Cluster phase 2: nobody leaves while a peer may still be reading its staging rows or
    // writing into its merge buffer (an owner arrives only after all its rows have landed).
    FALCON_TRACE(tid == 0, 75);
    cluster_arrive_relaxed();
    cluster_wait();
    FALCON_TRACE(tid == 0, 76);
  }
  if (warp == kWarpMma) {
    if (n_my > 0 && *abort_flag && lane == 0) {
      // after a wait that gave up, MMAs may still be running: the last commit covers them all
      for (uint32_t it = 0; it < (1u << 20); ++it) {
        uint32_t ok;
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                     : "=r"(ok)
                     : "r"(bar(kBarODone)), "r"(0u)
                     : "memory");
        if (ok) break;
      }
    }
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}


bool is_pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }

// Largest cluster size (number of KV splits) for which `units` clusters are co-resident.
int pick_splits(falcon_ctx* ctx, int units, int max_tiles) {
  // (both instantiations of the kernel have the same footprint: one CTA per SM)
  int* resident = ctx->attn_resident[0];
  int best = 1;
  for (int s = kMaxSplits; s >= 1; --s) {
    if (s > max_tiles) continue;
    if (resident[s] == 0) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(s, ctx->sm_count, 1);
      cfg.blockDim = dim3(kTcThreads);
      cfg.dynamicSmemBytes = kSmemAlloc;
      cudaLaunchAttribute attr;
      attr.id = cudaLaunchAttributeClusterDimension;
      attr.val.clusterDim.x = s;
      attr.val.clusterDim.y = 1;
      attr.val.clusterDim.z = 1;
      cfg.attrs = &attr;
      cfg.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, tree_attn_tc_kernel<false>, &cfg) != cudaSuccess) n = -1;
      resident[s] = n > 0 ? n : -1;
      cudaGetLastError();
    }
    if (resident[s] >= units) { best = s; break; }
  }
  return best;
}

}  // namespace

bool tree_attn_tc_supports(const falcon_ctx* ctx, const falcon_attn_args& a) {
  (void)ctx;
  if (a.head_dim != kD) return false;
  if (a.k_tree != nullptr) return false;
  if (!(a.sm_scale > 0.f)) return false;  // the kernel takes row maxima on unscaled scores
  const int G = a.n_q_heads / a.n_kv_heads;
  if (!is_pow2(G) || G > kBM) return false;
  if (a.n_splits > kMaxSplits) return false;
  if (a.tree.batch > 65535) return false;
  return get_encode() != nullptr;
}

int launch_tree_attn_tc(falcon_ctx* ctx, const falcon_attn_args& a, cudaStream_t s) {
  const int B = a.tree.batch, Hq = a.n_q_heads, Hkv = a.n_kv_heads, G = Hq / Hkv;
  const int n_mtiles = (a.tree.max_tree * G + kBM - 1) / kBM;
  if (static_cast<int64_t>(Hkv) * n_mtiles > 65535) return FALCON_ERR_CAPACITY;

  bool& attr_set = ctx->attn_attr_set[0];
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(tree_attn_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(kSmemAlloc));
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(tree_attn_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               static_cast<int>(kSmemAlloc));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaFuncSetAttribute(tree_attn_tc_kernel)");
    attr_set = true;
  }

  // Tensor maps.  The head dimension is split into (64 columns, 2 halves) so that one box covers both
  // 128-byte-swizzled half tiles.  K/V cache: [64, s_cap, 2, Hkv, B], box 64 x 64 keys x 2.
  uint64_t kv_dims[5] = {64, static_cast<uint64_t>(a.s_cap), 2, static_cast<uint64_t>(Hkv), static_cast<uint64_t>(B)};
  uint64_t kv_strides[4] = {static_cast<uint64_t>(a.kv_stride_s) * 2, 128, static_cast<uint64_t>(a.kv_stride_h) * 2,
                            static_cast<uint64_t>(a.kv_stride_b) * 2};
  if (Hkv == 1 && kv_strides[2] == 0) kv_strides[2] = kv_strides[0] * a.s_cap;  // a size-1 dimension never strides
  if (B == 1 && kv_strides[3] == 0) kv_strides[3] = kv_strides[2] * Hkv;
  const uint32_t kv_box[5] = {64, static_cast<uint32_t>(kBN), 2, 1, 1};
  const int max_tiles = (a.tree.max_prefix_len + a.tree.max_tree + kBN - 1) / kBN;
  int splits = a.n_splits;
  if (splits == 0) splits = pick_splits(ctx, Hkv * n_mtiles * B, max_tiles > 0 ? max_tiles : 1);
  if (splits < 1) splits = 1;
  // Trees of at most 64 query rows per KV head are held twice in the tile (two key-column groups per
  // row), unless the cluster is so large that the merge could not take twice as many partial results.
  const bool dup = a.tree.max_tree * G <= 64 && 2 * splits <= kMaxSplits;

  // q: [64, G, Hkv, N, 2]; a box is the query rows of one KV head: q_nodes nodes x G heads (at most
  // 128 rows, a multiple of 8 so that the second half starts on a swizzle-atom boundary).  With two
  // copies a box is one 64-column half of at most 64 rows, and each copy and half is its own load.
  const uint64_t row_bytes = static_cast<uint64_t>(kD) * 2;
  int q_nodes = kBM / G;
  {
    const int gran = G >= 8 ? 1 : 8 / G;
    const int want = (a.tree.max_tree + gran - 1) / gran * gran;
    if (want < q_nodes) q_nodes = want;
  }
  uint64_t q_dims[5] = {64, static_cast<uint64_t>(G), static_cast<uint64_t>(Hkv),
                        static_cast<uint64_t>(a.tree.total_nodes), 2};
  uint64_t q_strides[4] = {row_bytes, row_bytes * G, row_bytes * Hq, 128};
  const uint32_t q_box[5] = {64, static_cast<uint32_t>(G), 1, static_cast<uint32_t>(q_nodes), dup ? 1u : 2u};
  CUtensorMap mq, mk, mv;
  if (!get_tmap(ctx, a.q, q_dims, q_strides, q_box, &mq) || !get_tmap(ctx, a.k_cache, kv_dims, kv_strides, kv_box, &mk) ||
      !get_tmap(ctx, a.v_cache, kv_dims, kv_strides, kv_box, &mv)) {
    ctx->last_error = "cuTensorMapEncodeTiled failed";
    return FALCON_ERR_CUDA;
  }
  TcParams p;
  p.Hq = Hq;
  p.Hkv = Hkv;
  p.G = G;
  p.s_cap = a.s_cap;
  p.total_nodes = a.tree.total_nodes;
  p.scale_log2 = a.sm_scale * kLog2e;
  p.q_half_bytes = dup ? kBM * 128u : static_cast<uint32_t>(q_nodes) * G * 128u;
  p.q_box_bytes = static_cast<uint32_t>(q_nodes) * G * 128u * (dup ? 1u : 2u);
  p.node_off = a.tree.node_off;
  p.parent = a.tree.parent;
  p.prefix_len = a.tree.prefix_len;
  p.status = a.tree.status;
  p.tree_mask = a.tree_mask;
  p.have_host = 0;
  p.early_prefix = (a.flags & FALCON_ATTN_PREFIX_STABLE) ? 1 : 0;
  p.stall_first = (a.flags & FALCON_ATTN_TEST_STALL) ? 1 : 0;
  if (a.tree.prefix_len_host && a.tree.node_off_host && B <= kHostSeqs) {
    p.have_host = 1;
    for (int i = 0; i <= B; ++i) p.h_node_off[i] = a.tree.node_off_host[i];
    for (int i = 0; i < B; ++i) p.h_prefix[i] = a.tree.prefix_len_host[i];
  }
  p.q = static_cast<const __nv_bfloat16*>(a.q);
  p.out = static_cast<__nv_bfloat16*>(a.out);

  FALCON_TRACE_LAUNCH(p)

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(splits, Hkv * n_mtiles, B);
  cfg.blockDim = dim3(kTcThreads);
  cfg.dynamicSmemBytes = kSmemAlloc;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = splits;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  // Programmatic dependent launch: this grid may be scheduled while the previous kernel of the stream
  // drains; the kernel itself waits for that kernel's completion before it touches global memory.
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  cudaError_t e = dup ? cudaLaunchKernelEx(&cfg, tree_attn_tc_kernel<true>, mq, mk, mv, p)
                      : cudaLaunchKernelEx(&cfg, tree_attn_tc_kernel<false>, mq, mk, mv, p);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "tree_attn_tc_kernel launch");
  return FALCON_OK;
}

void tree_attn_tc_release(falcon_ctx* ctx) { release_tmaps(ctx); }

}  // namespace falcon
