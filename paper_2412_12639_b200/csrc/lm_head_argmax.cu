// falcon_lm_head_argmax: the greedy token of every tree node straight from the LM head
// (Section 3.1: the LM head turns the aggregated features into the distribution over the
// vocabulary; Eq. 6: p = Softmax(LM(f)); temperature 0, Section 4.1, needs only the position of the
// largest logit).  logit[i, v] = sum_k feat[i, k] * head[v, k] is a dense bf16 contraction whose
// [N, V] fp32 result is never written: the argmax is taken where the accumulator is read.
//
// The head (V x hidden bf16, 262 MB at 32000 x 4096) is read once and dominates: the kernel is
// bound by HBM, the tensor core is about a third busy.  Every CTA owns a run of vocabulary rows
// (V split evenly over the SMs, in steps of 16, so one launch is one wave) and streams it through a
// TMA ring in chunks of 64 hidden columns together with the matching chunk of the features (L2
// hits after the first CTA).  tcgen05.mma with the nodes on the M side (128 per tile; up to two
// tiles resident, so up to 256 nodes read the head once) and the CTA's vocabulary rows on the N
// side (up to 256 per instruction) accumulates in TMEM; four warps then read one accumulator row
// (= one node) each, 32 columns at a time, and keep the first maximum.  A CTA's result for a node
// is one 64-bit atomicMax on a word ordered by (logit, then lower index), so ties go to the lowest
// index whatever the timing; the last CTA to arrive unpacks the words.
//
// Warp roles: 0 = TMA producer (one thread), 1 = MMA issuer (one elected thread) and TMEM owner,
// 2-5 = accumulator readers.  Every wait is bounded; a wait that gives up sets FALCON_DEV_TIMEOUT
// in the caller's status word and the kernel still leaves in order (loads drained, MMAs finished,
// TMEM freed).

#include <climits>

#include "tc_util.cuh"

namespace falcon {
namespace {
using namespace tc;

constexpr int kLmThreads = 192;
constexpr int kLmReaders = 128;
constexpr int kLmKC = 64;             // hidden columns per ring stage: one 128-byte swizzle row of bf16
constexpr int kLmMaxStages = 8;
constexpr int kLmTileMax = 256;       // vocabulary rows per MMA (the N side) at most
constexpr uint32_t kLmSmemMax = 232448;
constexpr uint32_t kLmFeatPad = 64u * kLmKC * 2u;    // see f_rows: what a 64-row feature tile leaves for the MMA to read past

enum LmBar {
  kLmBarFull = 0,                            // [kLmMaxStages] a stage's tiles have landed
  kLmBarEmpty = kLmBarFull + kLmMaxStages,   // [kLmMaxStages] the MMAs that read a stage have finished
  kLmBarAccFull = kLmBarEmpty + kLmMaxStages,
  kLmBarAccEmpty,
  kLmBarDone,
  kLmNumBars
};
constexpr uint32_t kLmSmallBytes = kLmFeatPad + 8u * kLmNumBars + 16u;  // pad, barriers, TMEM base, abort flag, last-CTA flag

struct LmParams {
  int32_t n_rows, vocab;
  int32_t n_kc;       // 64-column chunks of the hidden dimension = ceil(hidden / 64)
  int32_t kch;        // chunks per ring stage
  int32_t f_rows;     // rows of a feature tile as loaded: 128, or with a single tile the number of nodes rounded up
                      // to 8 (64 at least); the MMA still reads 128 rows, and what follows the tile gives
                      // accumulator rows that nobody looks at
  int32_t n_mt;       // 128-node tiles
  int32_t m_res;      // node tiles resident in TMEM at once (1 or 2)
  int32_t tile_n;     // vocabulary rows per MMA (multiple of 16)
  int32_t span;       // vocabulary rows per CTA (multiple of 16)
  int32_t n_stages;
  int32_t stall_first;  // test hook: the features of ring stage 0 are never requested (a bounded wait then runs out)
  uint32_t stage_bytes, idesc;
  int32_t* argmax_out;
  float* max_out;
  int32_t* status;
  unsigned long long* best;  // [n_rows] the nodes' best (logit, index) so far as one orderable word; zero between calls
  int* ticket;               // zero between calls
};

// (logit, index) as one word whose unsigned order is "larger logit first, then the lower index"; 0 = nothing.
__device__ __forceinline__ unsigned long long lm_pack(float x, int idx) {
  const uint32_t b = __float_as_uint(x + 0.f);  // -0 -> +0
  const uint32_t key = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
  return (static_cast<unsigned long long>(key) << 32) | static_cast<uint32_t>(~idx);
}
__device__ __forceinline__ float lm_unpack_val(unsigned long long w) {
  const uint32_t k = static_cast<uint32_t>(w >> 32);
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

__device__ __forceinline__ bool lm_wait_drain(uint32_t bar, uint32_t parity) {
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

__global__ void __launch_bounds__(kLmThreads, 1)
lm_head_argmax_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_f, const LmParams p) {
  extern __shared__ __align__(1024) unsigned char smem_gen[];
  const uint32_t smem_base = smem_u32(smem_gen);
  unsigned char* small = smem_gen + static_cast<uint32_t>(p.n_stages) * p.stage_bytes + kLmFeatPad;
  const uint32_t bars = smem_u32(small);
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(small + 8 * kLmNumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(small + 8 * kLmNumBars + 4);
  volatile int* s_last = reinterpret_cast<volatile int*>(small + 8 * kLmNumBars + 8);
  auto bar = [&](int i) { return bars + 8u * static_cast<uint32_t>(i); };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cta = blockIdx.x, n_cta = gridDim.x;
  const int S = p.n_stages;
  const int v_lo = cta * p.span, v_hi = min(p.vocab, v_lo + p.span);
  const int n_vt = (v_hi - v_lo + p.tile_n - 1) / p.tile_n;  // >= 1 by construction of the grid
  const int n_groups = (p.n_mt + p.m_res - 1) / p.m_res;
  const uint32_t tmem_cols = static_cast<uint32_t>(p.m_res) * 256u;
  const uint32_t w_bytes = static_cast<uint32_t>(p.tile_n) * (kLmKC * 2u);   // one chunk of the head tile
  const uint32_t f_bytes = static_cast<uint32_t>(p.f_rows) * (kLmKC * 2u);   // one chunk of one feature tile
  const int n_ks = (p.n_kc + p.kch - 1) / p.kch;                             // ring stages per accumulator tile
  const int n_iter = n_groups * n_vt * n_ks;                                 // ring stages this CTA goes through
  const int n_pre = min(S, n_iter);
  // CTAs start at different places of the hidden dimension (a sum does not care where it starts), so that at
  // any moment they read different column ranges of their rows instead of all the same one.
  const int rot = static_cast<int>((static_cast<unsigned>(cta) * 11u) % static_cast<unsigned>(n_ks));
  // Ring stage `it` = (node-tile group, vocabulary tile, K step), K fastest.  Its chunks are asked for back to
  // back; a chunk past the hidden size reads as zeros, and so does a node tile past the last one.
  auto issue_head = [&](int it) {
    const int st = it % S, kq = (it % n_ks + rot) % n_ks, vt = (it / n_ks) % n_vt;
    const uint32_t dst = smem_base + static_cast<uint32_t>(st) * p.stage_bytes;
    for (int c = 0; c < p.kch; ++c)
      tma_load_5d(dst + c * w_bytes, &tm_w, bar(kLmBarFull + st), (kq * p.kch + c) * kLmKC, v_lo + vt * p.tile_n, 0, 0, 0);
  };
  auto issue_feat = [&](int it) {
    if (it == 0 && p.stall_first) return;
    const int st = it % S, kq = (it % n_ks + rot) % n_ks, g = it / (n_ks * n_vt);
    const uint32_t fdst = smem_base + static_cast<uint32_t>(st) * p.stage_bytes + static_cast<uint32_t>(p.kch) * w_bytes;
    for (int c = 0; c < p.kch; ++c)
      for (int j = 0; j < p.m_res; ++j)
        tma_load_5d(fdst + (c * p.m_res + j) * f_bytes, &tm_f, bar(kLmBarFull + st), (kq * p.kch + c) * kLmKC,
                    (g * p.m_res + j) * 128, 0, 0, 0);
  };

  if (warp == 0) {
    if (lane == 0) {
      *abort_flag = (smem_base & 1023u) ? 1 : 0;  // the swizzled tiles need a 1 KB aligned base
      *s_last = 0;
      prefetch_tmap(&tm_w);
      prefetch_tmap(&tm_f);
      for (int i = 0; i < kLmNumBars; ++i) mbar_init(bar(i), i == kLmBarAccEmpty ? kLmReaders / 32 : 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      // The head is a constant of the model: its first ring fill is asked for before the wait below, while
      // the previous kernel of the stream is still finishing.  The features are that kernel's to write.
      if (!*abort_flag)
        for (int it = 0; it < n_pre; ++it) {
          mbar_expect_tx(bar(kLmBarFull + it), p.stage_bytes);
          issue_head(it);
        }
    }
    __syncwarp();
  } else if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem_base)), "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // Under programmatic dependent launch the grid may start while the previous kernel of the stream
  // drains: the features (and the scratch) are that kernel's business until it has completed.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem_base;

  if (warp == 0) {
    // ================================ TMA producer ================================
    if (lane == 0) {
      bool ok = !*abort_flag;
      int it = ok ? n_pre : 0;
      if (ok)
        for (int i = 0; i < n_pre; ++i) issue_feat(i);
      for (; ok && it < n_iter; ++it) {
        const int st = it % S;
        ok = mbar_wait(bar(kLmBarEmpty + st), (it / S - 1) & 1, abort_flag);
        if (!ok) break;
        mbar_expect_tx(bar(kLmBarFull + st), p.stage_bytes);
        issue_head(it);
        issue_feat(it);
      }
      if (!ok || *abort_flag) {
        // Some wait gave up.  The tiles asked for still arrive: stay until they have, so that no copy
        // is in flight into this CTA's shared memory when it leaves.
        for (int j = max(0, it - S); j < it; ++j) lm_wait_drain(bar(kLmBarFull + j % S), (j / S) & 1);
      }
    }
  } else if (warp == 1) {
    // ================================ MMA issuer ================================
    uint32_t elected;
    asm volatile("{ .reg .pred p; elect.sync _|p, 0xffffffff; selp.u32 %0, 1, 0, p; }" : "=r"(elected));
    int it = 0, tile = 0;
    bool ok = !*abort_flag;
    for (int g = 0; ok && g < n_groups; ++g) {
      for (int vt = 0; ok && vt < n_vt; ++vt, ++tile) {
        if (tile > 0) ok = mbar_wait_warp(bar(kLmBarAccEmpty), (tile - 1) & 1, abort_flag);  // the readers are done with TMEM
        if (!ok) break;
        tc_fence_after();
        for (int ks = 0; ok && ks < n_ks; ++ks, ++it) {
          const int st = it % S;
          ok = mbar_wait_warp(bar(kLmBarFull + st), (it / S) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          if (elected) {
            const uint32_t wbase = smem_base + static_cast<uint32_t>(st) * p.stage_bytes;
            const uint32_t fbase = wbase + static_cast<uint32_t>(p.kch) * w_bytes;
            for (int c = 0; c < p.kch; ++c) {
              for (int j = 0; j < p.m_res; ++j) {
#pragma unroll
                for (int kk = 0; kk < kLmKC / 16; ++kk) {
                  // features (A) and head rows (B): both K-major, 16 hidden columns = 32 bytes inside the 128-byte swizzle row
                  const uint64_t ad = smem_desc(fbase + (c * p.m_res + j) * f_bytes + kk * 32, 16, 1024);
                  const uint64_t bd = smem_desc(wbase + c * w_bytes + kk * 32, 16, 1024);
                  umma_bf16_ss(tmem_base + static_cast<uint32_t>(j) * 256u, ad, bd, p.idesc, (ks > 0 || c > 0 || kk > 0) ? 1u : 0u);
                }
              }
            }
            umma_commit(bar(kLmBarEmpty + st));
          }
          __syncwarp();
        }
        if (ok && elected) umma_commit(bar(kLmBarAccFull));
        __syncwarp();
      }
    }
    // every MMA issued so far has finished before TMEM is given back
    if (elected) {
      umma_commit(bar(kLmBarDone));
      lm_wait_drain(bar(kLmBarDone), 0);
    }
    __syncwarp();
  } else {
    // ================================ accumulator readers ================================
    const int q = warp & 3;                 // TMEM lane quadrant this warp can reach
    const int r = q * 32 + lane;            // accumulator row = node inside its tile
    const int rt = tid - 64;                // 0 .. 127
    const uint32_t tmem_lane = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    int tile = 0;
    bool ok = !*abort_flag;
    for (int g = 0; g < n_groups; ++g) {
      float best[2] = {-INFINITY, -INFINITY};
      int idx[2] = {INT_MAX, INT_MAX};
      for (int vt = 0; ok && vt < n_vt; ++vt, ++tile) {
        ok = mbar_wait_warp(bar(kLmBarAccFull), tile & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const int v0 = v_lo + vt * p.tile_n;
        const int ncols = min(p.tile_n, v_hi - v0);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          if (j >= p.m_res) break;
          for (int c0 = 0; c0 < ncols; c0 += 32) {
            uint32_t x[32];
            FALCON_TMEM_LD32(tmem_lane + static_cast<uint32_t>(j) * 256u + static_cast<uint32_t>(c0), x);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              const float f = __uint_as_float(x[c]);
              if (c0 + c < ncols && f > best[j]) {  // strict: columns ascend, so the first maximum stays; NaN never wins
                best[j] = f;
                idx[j] = v0 + c0 + c;
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(kLmBarAccEmpty));
      }
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int node = (g * p.m_res + j) * 128 + r;
        // one atomic per node and CTA: the order of arrival does not matter, the word's order decides
        if (j < p.m_res && node < p.n_rows && ok && idx[j] != INT_MAX) atomicMax(p.best + node, lm_pack(best[j], idx[j]));
      }
    }
    // the last CTA to arrive folds the CTAs' results in vocabulary order
    asm volatile("bar.sync 1, %0;" ::"n"(kLmReaders) : "memory");
    if (rt == 0) {
      if (*abort_flag) dev_status_or(p.status, 0, FALCON_DEV_TIMEOUT);
      __threadfence();
      *s_last = (atomicAdd(p.ticket, 1) == n_cta - 1) ? 1 : 0;
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kLmReaders) : "memory");
    if (*s_last) {
      __threadfence();
      for (int node = rt; node < p.n_rows; node += kLmReaders) {
        const unsigned long long w = __ldcg(p.best + node);
        p.best[node] = 0ull;  // ready for the next call
        p.argmax_out[node] = w ? static_cast<int>(~static_cast<uint32_t>(w)) : 0;
        if (p.max_out) p.max_out[node] = w ? lm_unpack_val(w) : -INFINITY;
      }
      if (rt == 0) *p.ticket = 0;  // ready for the next call
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

}  // namespace

int launch_lm_head_argmax(falcon_ctx* ctx, const falcon_lm_argmax_args& a, cudaStream_t s) {
  const int N = a.n_rows, V = a.vocab, H = a.hidden;
  const int n_mt = (N + 127) / 128;
  const int m_res = n_mt >= 2 ? 2 : 1;
  // One wave: the vocabulary split evenly over the SMs in steps of 16 rows.
  int span = ((V + ctx->sm_count - 1) / ctx->sm_count + 15) & ~15;
  const int n_cta = (V + span - 1) / span;
  const int tile_n = span < kLmTileMax ? span : kLmTileMax;
  const int f_rows = n_mt > 1 ? 128 : (N <= 64 ? 64 : ((N + 7) & ~7));
  const int n_kc = (H + kLmKC - 1) / kLmKC;
  // Chunks per stage: two where two such stages fit.  Fewer, larger stages mean fewer trips round the ring
  // (32000 x 4096, 60 nodes: 43 us with two chunks in three stages against 53 with one in five and 46 with
  // three in two; a head stored chunk by chunk so that a tile is contiguous made no difference).
  const uint32_t chunk_bytes = (static_cast<uint32_t>(tile_n) + static_cast<uint32_t>(m_res * f_rows)) * (kLmKC * 2u);
  int kch = (2 * 2 * chunk_bytes <= kLmSmemMax - kLmSmallBytes) ? 2 : 1;
  if (kch > n_kc) kch = n_kc;
  const uint32_t stage_bytes = static_cast<uint32_t>(kch) * chunk_bytes;
  int n_stages = static_cast<int>((kLmSmemMax - kLmSmallBytes) / stage_bytes);
  if (n_stages > kLmMaxStages) n_stages = kLmMaxStages;
  if (n_stages < 2) return FALCON_ERR_CAPACITY;
  const uint32_t smem_bytes = static_cast<uint32_t>(n_stages) * stage_bytes + kLmSmallBytes;


  if (!ctx->lm_attr_set) {
    cudaError_t e = cudaFuncSetAttribute(lm_head_argmax_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(kLmSmemMax));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaFuncSetAttribute(lm_head_argmax_kernel)");
    ctx->lm_attr_set = true;
  }
  // scratch that is zero between calls: the arrival counter and one 64-bit word per node
  int rc = ensure_tickets(ctx, 2 + 2 * N, s);
  if (rc) return rc;

  // Tensor maps: [hidden, rows] with the hidden index contiguous; a box is 64 columns x the tile's
  // rows, 128-byte swizzled; what lies outside (the hidden tail, rows past the end) reads as zeros.
  CUtensorMap mw, mf;
  {
    const uint64_t hs = static_cast<uint64_t>(a.head_stride) * 2, fs = static_cast<uint64_t>(a.feat_stride) * 2;
    const uint64_t w_dims[5] = {static_cast<uint64_t>(H), static_cast<uint64_t>(V), 1, 1, 1};
    const uint64_t w_strides[4] = {hs, hs * V, hs * V, hs * V};
    const uint32_t w_box[5] = {kLmKC, static_cast<uint32_t>(tile_n), 1, 1, 1};
    const uint64_t f_dims[5] = {static_cast<uint64_t>(H), static_cast<uint64_t>(N), 1, 1, 1};
    const uint64_t f_strides[4] = {fs, fs * N, fs * N, fs * N};
    const uint32_t f_box[5] = {kLmKC, static_cast<uint32_t>(f_rows), 1, 1, 1};
    if (!get_tmap(ctx, a.lm_head, w_dims, w_strides, w_box, &mw) || !get_tmap(ctx, a.features, f_dims, f_strides, f_box, &mf)) {
      ctx->last_error = "cuTensorMapEncodeTiled failed";
      return FALCON_ERR_CUDA;
    }
  }

  LmParams p;
  p.n_rows = N;
  p.vocab = V;
  p.n_kc = n_kc;
  p.kch = kch;
  p.f_rows = f_rows;
  p.n_mt = n_mt;
  p.m_res = m_res;
  p.tile_n = tile_n;
  p.span = span;
  p.n_stages = n_stages;
  p.stall_first = (a.flags & FALCON_LM_TEST_STALL) ? 1 : 0;
  p.stage_bytes = stage_bytes;
  p.idesc = make_idesc(128, static_cast<uint32_t>(tile_n), false, false);
  p.argmax_out = a.argmax_out;
  p.max_out = a.max_out;
  p.status = a.status;
  p.ticket = ctx->tickets;
  p.best = reinterpret_cast<unsigned long long*>(ctx->tickets + 2);

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_cta);
  cfg.blockDim = dim3(kLmThreads);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, lm_head_argmax_kernel, mw, mf, p);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "lm_head_argmax_kernel launch");
  return FALCON_OK;
}

}  // namespace falcon
