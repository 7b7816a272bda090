// falcon_tree_attn, one small thread block per query row: the kernel for small problems (up to 1024
// keys a sequence, any head_dim the call supports, separate tree buffers, any head grouping), where
// a launch is a few microseconds of latency whatever the arithmetic costs and the tensor-core
// kernels' set-up is most of their time.  What counts here is the number of dependent round trips
// to memory, so every pass issues all its loads before it uses any.
//
// A block of four warps owns one (node, query head).  Pass 1: the 128 threads take the keys round
// robin, each thread reads its key's whole row (16-byte loads) and forms the score against the
// query (in shared memory, broadcast reads); masked keys (tree mask from the node's ancestor bit
// set) get -inf; the scores go to shared memory.  The row maximum and the sum of the weights are
// block reductions, so the softmax is the plain two-pass one in fp32.  Pass 2: each warp takes a
// quarter of the keys, its lanes the head dimensions (2 or 4 each), sixteen keys' loads in flight
// at a time; the four partial rows are added through shared memory.  Nothing is rounded before the
// final bf16.
#include "common.cuh"

namespace falcon {
namespace {

constexpr int kWarpsPerCta = 4;
constexpr int kWarpKeysMax = 1024;  // keys per sequence this kernel takes (scores live in shared memory)
constexpr int kWarpHostSeqs = 8;    // sequences whose scalars travel in the kernel's parameters

struct WarpParams {
  int32_t batch, Hq, Hkv, s_cap;
  float scale_log2;
  int64_t stride_b, stride_h, stride_s;
  const int32_t* node_off;
  const int32_t* parent;
  const int32_t* prefix_len;
  int32_t* status;
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  const __nv_bfloat16* k_cache;
  const __nv_bfloat16* v_cache;
  const __nv_bfloat16* k_tree;
  const __nv_bfloat16* v_tree;
  const uint64_t* tree_mask;
  int32_t have_host;  // the caller's host copies of the per-sequence scalars came with the call
  int32_t h_node_off[kWarpHostSeqs + 1];
  int32_t h_prefix[kWarpHostSeqs];
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int D>
__global__ void __launch_bounds__(32 * kWarpsPerCta) tree_attn_warp_kernel(const WarpParams p) {
  constexpr int kPerLane = D / 32;  // head dimensions per lane in pass 2
  constexpr int kThreads = 32 * kWarpsPerCta;
  __shared__ __align__(16) float q_s[D];
  __shared__ float s_s[kWarpKeysMax];
  __shared__ float red_s[2][kWarpsPerCta];
  __shared__ float acc_s[kWarpsPerCta][D];
  __shared__ int32_t par_s[FALCON_T_MAX];

  // Under programmatic dependent launch the grid may start while the previous kernel of the stream
  // drains: nothing is read or written before that kernel has completed.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int h = blockIdx.x, node = blockIdx.y, b = blockIdx.z;
  // With the caller's host copies of the per-sequence scalars nothing has to be fetched before the
  // addresses are known, and the query row, the tree's parent array and every thread's first key are
  // asked for together: one round trip instead of a chain (scalars, then parents one by one, then keys).
  int base, T_real, L_raw;
  if (p.have_host) {
    base = p.h_node_off[b];
    T_real = p.h_node_off[b + 1] - base;
    L_raw = p.h_prefix[b];
  } else {
    base = p.node_off[b];
    T_real = p.node_off[b + 1] - base;
    L_raw = p.prefix_len[b];
  }
  const int T = min(T_real, FALCON_T_MAX);
  if (node >= T) return;  // the whole block
  const int L = max(L_raw, 0);
  const bool separate = (p.k_tree != nullptr);
  const int prefix_rows = min(L, p.s_cap);
  const int S = min(separate ? prefix_rows + T : min(L + T, p.s_cap), kWarpKeysMax);
  const int G = p.Hq / p.Hkv, kvh = h / G;

  const __nv_bfloat16* kb = p.k_cache + b * p.stride_b + kvh * p.stride_h;
  const __nv_bfloat16* vb = p.v_cache + b * p.stride_b + kvh * p.stride_h;
  auto row_of = [&](const __nv_bfloat16* cache, const __nv_bfloat16* tree, int key) -> const __nv_bfloat16* {
    if (separate && key >= prefix_rows)
      return tree + (static_cast<int64_t>(base + key - prefix_rows) * p.Hkv + kvh) * D;
    return cache + static_cast<int64_t>(key) * p.stride_s;
  };

  const __nv_bfloat16* qrow = p.q + (static_cast<int64_t>(base + node) * p.Hq + h) * D;
  __nv_bfloat16 q_raw = __float2bfloat16(0.f);
  if (tid < D) q_raw = qrow[tid];
  int par_raw = -1;
  if (!p.tree_mask && tid < T) par_raw = p.parent[base + tid];
  uint4 kx0[D / 8];
  if (tid < S) {  // (masked or not: which tree keys count is known only after the walk below)
    const uint4* kr = reinterpret_cast<const uint4*>(row_of(kb, p.k_tree, tid));
#pragma unroll
    for (int c = 0; c < D / 8; ++c) kx0[c] = kr[c];
  }
  if (tid < D) q_s[tid] = __bfloat162float(q_raw);
  if (tid < T) par_s[tid] = par_raw;
  __syncthreads();

  uint64_t lo, hi;
  bool bad = false;
  if (p.tree_mask) {
    lo = p.tree_mask[2 * static_cast<int64_t>(base + node)];
    hi = p.tree_mask[2 * static_cast<int64_t>(base + node) + 1];
  } else {
    bad = !ancestor_mask(par_s, T, node, lo, hi);  // the walk, in shared memory
    if (node == 0 && par_s[0] != -1) bad = true;
  }
  if (tid == 0 && h == 0) {
    if (bad) dev_status_or(p.status, b, FALCON_DEV_BAD_TREE);
    if (node == 0 && (L + (separate ? 0 : T) > p.s_cap || T_real > FALCON_T_MAX || L + T > kWarpKeysMax))
      dev_status_or(p.status, b, FALCON_DEV_CAPACITY);
  }

  // ---- pass 1: scores (one key per thread and round), row maximum ----
  auto score = [&](const uint4 (&kx)[D / 8]) -> float {
    float acc = 0.f;
#pragma unroll
    for (int c = 0; c < D / 8; ++c) {
      const float4 qa = *reinterpret_cast<const float4*>(&q_s[8 * c]);
      const float4 qb = *reinterpret_cast<const float4*>(&q_s[8 * c + 4]);
      const __nv_bfloat162* kh = reinterpret_cast<const __nv_bfloat162*>(&kx[c]);
      const float2 k0 = __bfloat1622float2(kh[0]), k1 = __bfloat1622float2(kh[1]);
      const float2 k2 = __bfloat1622float2(kh[2]), k3 = __bfloat1622float2(kh[3]);
      acc = fmaf(qa.x, k0.x, acc);
      acc = fmaf(qa.y, k0.y, acc);
      acc = fmaf(qa.z, k1.x, acc);
      acc = fmaf(qa.w, k1.y, acc);
      acc = fmaf(qb.x, k2.x, acc);
      acc = fmaf(qb.y, k2.y, acc);
      acc = fmaf(qb.z, k3.x, acc);
      acc = fmaf(qb.w, k3.y, acc);
    }
    return acc * p.scale_log2;
  };
  float mx = -INFINITY;
  if (tid < S) {  // this thread's first key is in registers already
    const float s = (tid < prefix_rows || bit128(lo, hi, tid - prefix_rows)) ? score(kx0) : -INFINITY;
    s_s[tid] = s;
    mx = s;
  }
  for (int key = tid + kThreads; key < S; key += kThreads) {
    float s = -INFINITY;
    if (key < prefix_rows || bit128(lo, hi, key - prefix_rows)) {
      const uint4* kr = reinterpret_cast<const uint4*>(row_of(kb, p.k_tree, key));
      uint4 kx[D / 8];
#pragma unroll
      for (int c = 0; c < D / 8; ++c) kx[c] = kr[c];
      s = score(kx);
    }
    s_s[key] = s;
    mx = fmaxf(mx, s);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (lane == 0) red_s[0][warp] = mx;
  __syncthreads();
  mx = fmaxf(fmaxf(red_s[0][0], red_s[0][1]), fmaxf(red_s[0][2], red_s[0][3]));

  // ---- weights and their sum ----
  float sum = 0.f;
  for (int key = tid; key < S; key += kThreads) {
    const float s = s_s[key];
    const float w = (s == -INFINITY || mx == -INFINITY) ? 0.f : ex2f(s - mx);
    s_s[key] = w;
    sum += w;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (lane == 0) red_s[1][warp] = sum;
  __syncthreads();
  sum = (red_s[1][0] + red_s[1][1]) + (red_s[1][2] + red_s[1][3]);

  // ---- pass 2: out = sum_key w[key] . V[key]; this warp's quarter of the keys, this lane's head
  // dimensions.  Sixteen keys a round, their loads issued together; a key of weight zero (masked)
  // contributes nothing whatever its row holds, NaN included. ----
  float acc[kPerLane];
#pragma unroll
  for (int i = 0; i < kPerLane; ++i) acc[i] = 0.f;
  const int per_warp = (S + kWarpsPerCta - 1) / kWarpsPerCta;
  const int kbeg = warp * per_warp, kend = min(S, kbeg + per_warp);
  for (int k0 = kbeg; k0 < kend; k0 += 16) {
    float w[16];
    uint2 raw[16];
#pragma unroll
    for (int u = 0; u < 16; ++u) {
      const int key = min(k0 + u, kend - 1);
      w[u] = (k0 + u < kend) ? s_s[key] : 0.f;
      const __nv_bfloat16* vr = row_of(vb, p.v_tree, key) + lane * kPerLane;
      if constexpr (kPerLane == 2) {
        raw[u].x = *reinterpret_cast<const uint32_t*>(vr);
        raw[u].y = 0u;
      } else {
        raw[u] = *reinterpret_cast<const uint2*>(vr);
      }
    }
#pragma unroll
    for (int u = 0; u < 16; ++u) {
      const bool on = w[u] != 0.f;
      const float2 v0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw[u].x));
      acc[0] = fmaf(w[u], on ? v0.x : 0.f, acc[0]);
      acc[1] = fmaf(w[u], on ? v0.y : 0.f, acc[1]);
      if constexpr (kPerLane == 4) {
        const float2 v1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw[u].y));
        acc[2] = fmaf(w[u], on ? v1.x : 0.f, acc[2]);
        acc[3] = fmaf(w[u], on ? v1.y : 0.f, acc[3]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < kPerLane; ++i) acc_s[warp][lane * kPerLane + i] = acc[i];
  __syncthreads();
  if (tid < D) {
    const float inv = sum > 0.f ? 1.f / sum : 0.f;
    const float o = (acc_s[0][tid] + acc_s[1][tid]) + (acc_s[2][tid] + acc_s[3][tid]);
    p.out[(static_cast<int64_t>(base + node) * p.Hq + h) * D + tid] = __float2bfloat16_rn(o * inv);
  }
}

}  // namespace

bool tree_attn_warp_supports(const falcon_ctx* ctx, const falcon_attn_args& a) {
  (void)ctx;
  return a.tree.max_prefix_len + a.tree.max_tree <= kWarpKeysMax && a.tree.batch <= 65535 && a.n_q_heads <= 65535;
}

int launch_tree_attn_warp(falcon_ctx* ctx, const falcon_attn_args& a, cudaStream_t s) {
  WarpParams p;
  p.batch = a.tree.batch;
  p.Hq = a.n_q_heads;
  p.Hkv = a.n_kv_heads;
  p.s_cap = a.s_cap;
  p.scale_log2 = a.sm_scale * kLog2e;
  p.stride_b = a.kv_stride_b;
  p.stride_h = a.kv_stride_h;
  p.stride_s = a.kv_stride_s;
  p.node_off = a.tree.node_off;
  p.parent = a.tree.parent;
  p.prefix_len = a.tree.prefix_len;
  p.status = a.tree.status;
  p.q = static_cast<const __nv_bfloat16*>(a.q);
  p.out = static_cast<__nv_bfloat16*>(a.out);
  p.k_cache = static_cast<const __nv_bfloat16*>(a.k_cache);
  p.v_cache = static_cast<const __nv_bfloat16*>(a.v_cache);
  p.k_tree = static_cast<const __nv_bfloat16*>(a.k_tree);
  p.v_tree = static_cast<const __nv_bfloat16*>(a.v_tree);
  p.tree_mask = a.tree_mask;
  p.have_host = 0;
  if (a.tree.prefix_len_host && a.tree.node_off_host && a.tree.batch <= kWarpHostSeqs) {
    p.have_host = 1;
    for (int i = 0; i <= a.tree.batch; ++i) p.h_node_off[i] = a.tree.node_off_host[i];
    for (int i = 0; i < a.tree.batch; ++i) p.h_prefix[i] = a.tree.prefix_len_host[i];
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(a.n_q_heads, a.tree.max_tree, a.tree.batch);
  cfg.blockDim = dim3(32 * kWarpsPerCta);
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  const cudaError_t e = a.head_dim == 128 ? cudaLaunchKernelEx(&cfg, tree_attn_warp_kernel<128>, p)
                                          : cudaLaunchKernelEx(&cfg, tree_attn_warp_kernel<64>, p);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "tree_attn_warp_kernel launch");
  return FALCON_OK;
}

}  // namespace falcon
