// falcon_lm_head_argmax: the greedy token of every tree node straight from the LM head
// (Section 3.1: "the LM Head computes the probability distribution based on the aggregated
// features"; Eq. 6: p = Softmax(LM(f)); temperature 0, Section 4.1, needs only the position of the
// largest logit).  logit[i, v] = sum_k feat[i, k] * head[v, k] is a dense bf16 contraction whose
// [N, V] fp32 result is never written: the argmax is taken where the accumulator is read.
//
// The head (V x hidden bf16, 262 MB at 32000 x 4096) is read once and dominates: the kernel is
// bound by HBM, the tensor core is about a quarter busy.  Every CTA owns a run of vocabulary rows
// (V split evenly over the SMs, in steps of 16, so one launch is one wave) and streams it through a
// TMA ring in chunks of 64 hidden columns together with the matching chunk of the features (L2
// hits after the first CTA).  tcgen05.mma with the nodes on the M side (128 per tile; up to two
// tiles resident, so up to 256 nodes read the head once) and the CTA's vocabulary rows on the N
// side (up to 256 per instruction) accumulates in TMEM; four warps then read one accumulator row
// (= one node) each, 32 columns at a time, and keep the first maximum.  Per-CTA results go to
// scratch and the last CTA to arrive folds them in vocabulary order, so ties go to the lowest
// index whatever the timing.
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
constexpr uint32_t kLmFeatTile = 128u * kLmKC * 2u;  // bytes of one 128-node x 64-column feature tile

enum LmBar {
  kLmBarFull = 0,                            // [kLmMaxStages] a stage's tiles have landed
  kLmBarEmpty = kLmBarFull + kLmMaxStages,   // [kLmMaxStages] the MMAs that read a stage have finished
  kLmBarAccFull = kLmBarEmpty + kLmMaxStages,
  kLmBarAccEmpty,
  kLmBarDone,
  kLmNumBars
};
constexpr uint32_t kLmSmallBytes = 8u * kLmNumBars + 16u;  // barriers, TMEM base, abort flag, last-CTA flag

struct LmParams {
  int32_t n_rows, vocab;
  int32_t n_kc;       // ring stages per accumulator tile = ceil(hidden / 64)
  int32_t n_mt;       // 128-node tiles
  int32_t m_res;      // node tiles resident in TMEM at once (1 or 2)
  int32_t tile_n;     // vocabulary rows per MMA (multiple of 16)
  int32_t span;       // vocabulary rows per CTA (multiple of 16)
  int32_t n_stages;
  uint32_t stage_bytes, idesc;
  int32_t* argmax_out;
  float* max_out;
  int32_t* status;
  float* part_val;    // [n_rows, CTAs]
  int32_t* part_idx;  // [n_rows, CTAs]
  int* ticket;        // zero between calls
};

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
  unsigned char* small = smem_gen + static_cast<uint32_t>(p.n_stages) * p.stage_bytes;
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
  const uint32_t w_bytes = static_cast<uint32_t>(p.tile_n) * (kLmKC * 2u);

  if (warp == 0) {
    if (lane == 0) {
      *abort_flag = (smem_base & 1023u) ? 1 : 0;  // the swizzled tiles need a 1 KB aligned base
      *s_last = 0;
      prefetch_tmap(&tm_w);
      prefetch_tmap(&tm_f);
      for (int i = 0; i < kLmNumBars; ++i) mbar_init(bar(i), i == kLmBarAccEmpty ? kLmReaders / 32 : 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
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
      int it = 0;
      bool ok = !*abort_flag;
      for (int g = 0; ok && g < n_groups; ++g) {
        for (int vt = 0; ok && vt < n_vt; ++vt) {
          for (int kc = 0; ok && kc < p.n_kc; ++kc, ++it) {
            const int st = it % S;
            if (it >= S) ok = mbar_wait(bar(kLmBarEmpty + st), (it / S - 1) & 1, abort_flag);
            if (!ok) break;
            const uint32_t dst = smem_base + static_cast<uint32_t>(st) * p.stage_bytes;
            mbar_expect_tx(bar(kLmBarFull + st), p.stage_bytes);
            tma_load_5d(dst, &tm_w, bar(kLmBarFull + st), kc * kLmKC, v_lo + vt * p.tile_n, 0, 0, 0);
            for (int j = 0; j < p.m_res; ++j)  // (a node tile past the last one reads as zeros)
              tma_load_5d(dst + w_bytes + j * kLmFeatTile, &tm_f, bar(kLmBarFull + st), kc * kLmKC, (g * p.m_res + j) * 128, 0,
                          0, 0);
          }
        }
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
        for (int kc = 0; ok && kc < p.n_kc; ++kc, ++it) {
          const int st = it % S;
          ok = mbar_wait_warp(bar(kLmBarFull + st), (it / S) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          if (elected) {
            const uint32_t wbase = smem_base + static_cast<uint32_t>(st) * p.stage_bytes, fbase = wbase + w_bytes;
            for (int j = 0; j < p.m_res; ++j) {
#pragma unroll
              for (int kk = 0; kk < kLmKC / 16; ++kk) {
                // features (A) and head rows (B): both K-major, 16 hidden columns = 32 bytes inside the 128-byte swizzle row
                const uint64_t ad = smem_desc(fbase + j * kLmFeatTile + kk * 32, 16, 1024);
                const uint64_t bd = smem_desc(wbase + kk * 32, 16, 1024);
                umma_bf16_ss(tmem_base + static_cast<uint32_t>(j) * 256u, ad, bd, p.idesc, (kc > 0 || kk > 0) ? 1u : 0u);
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
        if (j < p.m_res && node < p.n_rows) {
          p.part_val[static_cast<int64_t>(node) * n_cta + cta] = ok ? best[j] : -INFINITY;
          p.part_idx[static_cast<int64_t>(node) * n_cta + cta] = ok ? idx[j] : INT_MAX;
        }
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
        float bv = -INFINITY;
        int bi = INT_MAX;
        const int64_t o = static_cast<int64_t>(node) * n_cta;
        for (int c = 0; c < n_cta; c += 8) {  // eight partials in flight: the loads are independent
          float v[8];
          int ix[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const bool in = c + k < n_cta;
            v[k] = in ? __ldcg(p.part_val + o + c + k) : -INFINITY;
            ix[k] = in ? __ldcg(p.part_idx + o + c + k) : INT_MAX;
          }
#pragma unroll
          for (int k = 0; k < 8; ++k)
            if (v[k] > bv) {  // CTAs ascend in vocabulary: strict keeps the lowest index
              bv = v[k];
              bi = ix[k];
            }
        }
        p.argmax_out[node] = bi == INT_MAX ? 0 : bi;
        if (p.max_out) p.max_out[node] = bv;
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
  const uint32_t stage_bytes = static_cast<uint32_t>(tile_n) * (kLmKC * 2u) + static_cast<uint32_t>(m_res) * kLmFeatTile;
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
  const size_t part = static_cast<size_t>(N) * n_cta;
  int rc = ensure_workspace(ctx, part * 8 + 256);
  if (rc) return rc;
  rc = ensure_tickets(ctx, 1, s);
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
    const uint32_t f_box[5] = {kLmKC, 128, 1, 1, 1};
    if (!get_tmap(ctx, a.lm_head, w_dims, w_strides, w_box, &mw) || !get_tmap(ctx, a.features, f_dims, f_strides, f_box, &mf)) {
      ctx->last_error = "cuTensorMapEncodeTiled failed";
      return FALCON_ERR_CUDA;
    }
  }

  LmParams p;
  p.n_rows = N;
  p.vocab = V;
  p.n_kc = (H + kLmKC - 1) / kLmKC;
  p.n_mt = n_mt;
  p.m_res = m_res;
  p.tile_n = tile_n;
  p.span = span;
  p.n_stages = n_stages;
  p.stage_bytes = stage_bytes;
  p.idesc = make_idesc(128, static_cast<uint32_t>(tile_n), false, false);
  p.argmax_out = a.argmax_out;
  p.max_out = a.max_out;
  p.status = a.status;
  p.part_val = static_cast<float*>(ctx->ws);
  p.part_idx = reinterpret_cast<int32_t*>(static_cast<float*>(ctx->ws) + part);
  p.ticket = ctx->tickets;

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
