// falcon_tree_attn, CUDA-core kernel: the path for shapes the tensor-core
// kernel does not take (head_dim 64, separate tree buffers, odd strides) and the
// on-GPU cross-check of that kernel.
//
// One CTA handles one (sequence, query head, KV split): it keeps the head's
// T x D queries in shared memory, walks its key range in tiles of 32 keys
// (16-byte coalesced loads into padded shared memory), computes the T x 32
// score tile with 4x4 register blocks, applies the tree mask from per-node
// ancestor bitmasks, runs an online softmax (one thread per node) and
// accumulates P.V in registers (4 nodes x D/4 columns per thread).  With more
// than one split the unnormalised partials go to scratch memory and the last
// CTA of the head (arrival counter) merges them.
#include "common.cuh"

namespace falcon {
namespace {

constexpr int kThreads = 128;
constexpr int kTileKeys = 32;
constexpr int kPad = 8;       // bf16 elements of row padding (16 bytes): conflict-free 16-byte row reads
constexpr int kSPitch = 33;   // floats per score row

struct SimtParams {
  int32_t batch, total_nodes, Hq, Hkv, s_cap, n_splits;
  float scale_log2;  // sm_scale * log2(e)
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
  float* part_o;    // [n_splits, N, Hq, D]
  float2* part_ml;  // [n_splits, N, Hq]
  int* tickets;     // [B * Hq]
};

__device__ __forceinline__ void unpack8(const uint4& u, float* f) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 t = __bfloat1622float2(h[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}

template <int D>
__global__ void __launch_bounds__(kThreads) tree_attn_simt_kernel(const SimtParams p) {
  constexpr int kPitch = D + kPad;  // bf16 elements per smem row
  constexpr int DB = D / 4;         // output columns per thread
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __nv_bfloat16* q_s = reinterpret_cast<__nv_bfloat16*>(smem_raw);              // [128][kPitch]
  __nv_bfloat16* k_s = q_s + FALCON_T_MAX * kPitch;                             // [32][kPitch]
  __nv_bfloat16* v_s = k_s + kTileKeys * kPitch;                                // [32][kPitch]
  float* s_s = reinterpret_cast<float*>(v_s + kTileKeys * kPitch);              // [128][33]
  uint64_t* anc_s = reinterpret_cast<uint64_t*>(s_s + FALCON_T_MAX * kSPitch);  // [128][2]
  float* m_s = reinterpret_cast<float*>(anc_s + 2 * FALCON_T_MAX);              // [128]
  float* l_s = m_s + FALCON_T_MAX;
  float* a_s = l_s + FALCON_T_MAX;
  __shared__ int s_last;

  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z, tid = threadIdx.x;
  const int G = p.Hq / p.Hkv, kvh = h / G;
  const int base = p.node_off[b];
  const int T = min(p.node_off[b + 1] - base, FALCON_T_MAX);
  const int L = max(p.prefix_len[b], 0);
  const bool separate = (p.k_tree != nullptr);
  // keys that can be read: in-cache tree rows must lie below s_cap
  const int prefix_rows = min(L, p.s_cap);
  const int S = separate ? prefix_rows + T : min(L + T, p.s_cap);

  // ---- per-node visibility masks --------------------------------------------------------------
  bool bad = false;
  if (tid < T) {
    uint64_t lo, hi;
    if (p.tree_mask) {
      lo = p.tree_mask[2 * static_cast<int64_t>(base + tid)];
      hi = p.tree_mask[2 * static_cast<int64_t>(base + tid) + 1];
    } else {
      bad = !ancestor_mask(p.parent + base, T, tid, lo, hi);
      if (tid == 0 && p.parent[base] != -1) bad = true;
    }
    anc_s[2 * tid] = lo;
    anc_s[2 * tid + 1] = hi;
  }
  m_s[tid] = -INFINITY;
  l_s[tid] = 0.f;
  if (bad && split == 0 && h == 0) dev_status_or(p.status, b, FALCON_DEV_BAD_TREE);
  if (tid == 0 && split == 0 && h == 0 &&
      (L + (separate ? 0 : T) > p.s_cap || p.node_off[b + 1] - base > FALCON_T_MAX))
    dev_status_or(p.status, b, FALCON_DEV_CAPACITY);

  // ---- queries of this head -------------------------------------------------------------------
  for (int idx = tid; idx < FALCON_T_MAX * (D / 8); idx += kThreads) {
    const int r = idx / (D / 8), c = idx % (D / 8);
    uint4 v = make_uint4(0, 0, 0, 0);
    if (r < T) v = *reinterpret_cast<const uint4*>(p.q + (static_cast<int64_t>(base + r) * p.Hq + h) * D + 8 * c);
    *reinterpret_cast<uint4*>(q_s + r * kPitch + 8 * c) = v;
  }

  // ---- key range of this split ----------------------------------------------------------------
  const int n_tiles = (S + kTileKeys - 1) / kTileKeys;
  const int tiles_per = (n_tiles + p.n_splits - 1) / p.n_splits;
  const int key_begin = min(S, split * tiles_per * kTileKeys);
  const int key_end = min(S, (split + 1) * tiles_per * kTileKeys);

  const __nv_bfloat16* kb = p.k_cache + b * p.stride_b + kvh * p.stride_h;
  const __nv_bfloat16* vb = p.v_cache + b * p.stride_b + kvh * p.stride_h;

  const int nb = tid >> 2, db = tid & 3;  // P.V ownership: nodes 4*nb.., columns DB*db..
  float acc[4][DB];
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int d = 0; d < DB; ++d) acc[r][d] = 0.f;
  const int TP4 = (T + 3) >> 2;  // node blocks in use

  for (int k0 = key_begin; k0 < key_end; k0 += kTileKeys) {
    __syncthreads();  // previous tile fully consumed (also orders the prologue writes)
    // -- load K and V tile --
    for (int idx = tid; idx < kTileKeys * (D / 8); idx += kThreads) {
      const int r = idx / (D / 8), c = idx % (D / 8);
      const int key = k0 + r;
      uint4 kx = make_uint4(0, 0, 0, 0), vx = kx;
      if (key < key_end) {
        if (separate && key >= prefix_rows) {
          const int64_t off = (static_cast<int64_t>(base + key - prefix_rows) * p.Hkv + kvh) * D + 8 * c;
          kx = *reinterpret_cast<const uint4*>(p.k_tree + off);
          vx = *reinterpret_cast<const uint4*>(p.v_tree + off);
        } else {
          kx = *reinterpret_cast<const uint4*>(kb + static_cast<int64_t>(key) * p.stride_s + 8 * c);
          vx = *reinterpret_cast<const uint4*>(vb + static_cast<int64_t>(key) * p.stride_s + 8 * c);
        }
      }
      *reinterpret_cast<uint4*>(k_s + r * kPitch + 8 * c) = kx;
      *reinterpret_cast<uint4*>(v_s + r * kPitch + 8 * c) = vx;
    }
    __syncthreads();

    // -- scores: 4 nodes x 4 keys per item --
    for (int item = tid; item < TP4 * (kTileKeys / 4); item += kThreads) {
      const int qn = item / (kTileKeys / 4), kq = item % (kTileKeys / 4);
      float s[4][4];
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) s[r][c] = 0.f;
#pragma unroll 2
      for (int d0 = 0; d0 < D; d0 += 8) {
        float qf[4][8], kf[4][8];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          unpack8(*reinterpret_cast<const uint4*>(q_s + (4 * qn + r) * kPitch + d0), qf[r]);
          unpack8(*reinterpret_cast<const uint4*>(k_s + (4 * kq + r) * kPitch + d0), kf[r]);
        }
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
          for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int d = 0; d < 8; ++d) s[r][c] = fmaf(qf[r][d], kf[c][d], s[r][c]);
      }
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int node = 4 * qn + r;
        const uint64_t lo = anc_s[2 * node], hi = anc_s[2 * node + 1];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int key = k0 + 4 * kq + c;
          bool vis = (node < T) && (key < key_end);
          if (vis && key >= prefix_rows)
            vis = (key - prefix_rows < FALCON_T_MAX) && bit128(lo, hi, key - prefix_rows);
          s_s[node * kSPitch + 4 * kq + c] = vis ? s[r][c] * p.scale_log2 : -INFINITY;
        }
      }
    }
    __syncthreads();

    // -- online softmax, one thread per node --
    if (tid < T) {
      float* row = s_s + tid * kSPitch;
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < kTileKeys; ++j) mx = fmaxf(mx, row[j]);
      const float m_old = m_s[tid];
      const float m_new = fmaxf(m_old, mx);
      float alpha = 1.f, sum = 0.f;
      if (m_new == -INFINITY) {
#pragma unroll
        for (int j = 0; j < kTileKeys; ++j) row[j] = 0.f;
      } else {
        alpha = exp2f(m_old - m_new);  // m_old = -inf gives 0
#pragma unroll
        for (int j = 0; j < kTileKeys; ++j) {
          const float e = exp2f(row[j] - m_new);
          row[j] = e;
          sum += e;
        }
      }
      m_s[tid] = m_new;
      l_s[tid] = l_s[tid] * alpha + sum;
      a_s[tid] = alpha;
    }
    __syncthreads();

    // -- O = alpha * O + P.V --
    if (nb < TP4) {
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const float al = (4 * nb + r < T) ? a_s[4 * nb + r] : 1.f;
#pragma unroll
        for (int d = 0; d < DB; ++d) acc[r][d] *= al;
      }
#pragma unroll 4
      for (int j = 0; j < kTileKeys; ++j) {
        float pj[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) pj[r] = (4 * nb + r < T) ? s_s[(4 * nb + r) * kSPitch + j] : 0.f;
#pragma unroll
        for (int d0 = 0; d0 < DB; d0 += 8) {
          float vf[8];
          unpack8(*reinterpret_cast<const uint4*>(v_s + j * kPitch + DB * db + d0), vf);
#pragma unroll
          for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int d = 0; d < 8; ++d) acc[r][d0 + d] = fmaf(pj[r], vf[d], acc[r][d0 + d]);
        }
      }
    }
  }
  __syncthreads();

  // ---- epilogue ---------------------------------------------------------------------------------
  if (p.n_splits == 1) {
    if (nb < TP4) {
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int node = 4 * nb + r;
        if (node >= T) continue;
        const float l = l_s[node];
        const float inv = l > 0.f ? 1.f / l : 0.f;
        __nv_bfloat16* o = p.out + (static_cast<int64_t>(base + node) * p.Hq + h) * D + DB * db;
#pragma unroll
        for (int d0 = 0; d0 < DB; d0 += 8) {
          __align__(16) __nv_bfloat162 pk[4];
#pragma unroll
          for (int d = 0; d < 4; ++d)
            pk[d] = __floats2bfloat162_rn(acc[r][d0 + 2 * d] * inv, acc[r][d0 + 2 * d + 1] * inv);
          *reinterpret_cast<uint4*>(o + d0) = *reinterpret_cast<const uint4*>(pk);
        }
      }
    }
    return;
  }

  // partials to scratch, then the last CTA of (b, h) merges
  const int64_t N = p.total_nodes;
  if (nb < TP4) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int node = 4 * nb + r;
      if (node >= T) continue;
      float* o = p.part_o + ((static_cast<int64_t>(split) * N + base + node) * p.Hq + h) * D + DB * db;
#pragma unroll
      for (int d0 = 0; d0 < DB; d0 += 4)
        __stcg(reinterpret_cast<float4*>(o + d0),
               make_float4(acc[r][d0], acc[r][d0 + 1], acc[r][d0 + 2], acc[r][d0 + 3]));
    }
  }
  if (tid < T)
    __stcg(p.part_ml + (static_cast<int64_t>(split) * N + base + tid) * p.Hq + h, make_float2(m_s[tid], l_s[tid]));
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int arrived = atomicAdd(&p.tickets[b * p.Hq + h], 1);
    s_last = (arrived == p.n_splits - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();

  if (nb < TP4) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int node = 4 * nb + r;
      if (node >= T) continue;
      float gm = -INFINITY;
      for (int s = 0; s < p.n_splits; ++s)
        gm = fmaxf(gm, __ldcg(p.part_ml + (static_cast<int64_t>(s) * N + base + node) * p.Hq + h).x);
      float lsum = 0.f, o[DB];
#pragma unroll
      for (int d = 0; d < DB; ++d) o[d] = 0.f;
      for (int s = 0; s < p.n_splits; ++s) {
        const float2 ml = __ldcg(p.part_ml + (static_cast<int64_t>(s) * N + base + node) * p.Hq + h);
        if (ml.x == -INFINITY) continue;
        const float w = exp2f(ml.x - gm);
        lsum += ml.y * w;
        const float* po = p.part_o + ((static_cast<int64_t>(s) * N + base + node) * p.Hq + h) * D + DB * db;
#pragma unroll
        for (int d0 = 0; d0 < DB; d0 += 4) {
          const float4 x = __ldcg(reinterpret_cast<const float4*>(po + d0));
          o[d0] = fmaf(x.x, w, o[d0]);
          o[d0 + 1] = fmaf(x.y, w, o[d0 + 1]);
          o[d0 + 2] = fmaf(x.z, w, o[d0 + 2]);
          o[d0 + 3] = fmaf(x.w, w, o[d0 + 3]);
        }
      }
      const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
      __nv_bfloat16* dst = p.out + (static_cast<int64_t>(base + node) * p.Hq + h) * D + DB * db;
#pragma unroll
      for (int d0 = 0; d0 < DB; d0 += 8) {
        __align__(16) __nv_bfloat162 pk[4];
#pragma unroll
        for (int d = 0; d < 4; ++d) pk[d] = __floats2bfloat162_rn(o[d0 + 2 * d] * inv, o[d0 + 2 * d + 1] * inv);
        *reinterpret_cast<uint4*>(dst + d0) = *reinterpret_cast<const uint4*>(pk);
      }
    }
  }
  if (tid == 0) p.tickets[b * p.Hq + h] = 0;
}

template <int D>
constexpr size_t simt_smem_bytes() {
  return static_cast<size_t>(FALCON_T_MAX + 2 * kTileKeys) * (D + kPad) * 2 + FALCON_T_MAX * kSPitch * 4 +
         FALCON_T_MAX * 16 + 3 * FALCON_T_MAX * 4;
}

}  // namespace

int launch_tree_attn_simt(falcon_ctx* ctx, const falcon_attn_args& a, cudaStream_t s) {
  const int B = a.tree.batch, Hq = a.n_q_heads;
  if (B > 65535 || Hq > 65535) return FALCON_ERR_CAPACITY;
  int splits = a.n_splits;
  const int max_keys = a.tree.max_prefix_len + a.tree.max_tree;
  const int n_tiles = (max_keys + kTileKeys - 1) / kTileKeys;
  if (splits == 0) {
    splits = (2 * ctx->sm_count + B * Hq - 1) / (B * Hq);
    // down to one 32-key tile per split: a tile costs this kernel several microseconds (measured),
    // far more than the merge of one more partial result
  }
  if (splits > 64) splits = 64;
  if (splits > n_tiles) splits = n_tiles;
  if (splits < 1) splits = 1;

  SimtParams p;
  p.batch = B;
  p.total_nodes = a.tree.total_nodes;
  p.Hq = Hq;
  p.Hkv = a.n_kv_heads;
  p.s_cap = a.s_cap;
  p.n_splits = splits;
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
  p.part_o = nullptr;
  p.part_ml = nullptr;
  p.tickets = nullptr;
  if (splits > 1) {
    const size_t rows = static_cast<size_t>(splits) * a.tree.total_nodes * Hq;
    const size_t o_bytes = rows * a.head_dim * sizeof(float);
    int rc = ensure_workspace(ctx, o_bytes + rows * sizeof(float2) + 256);
    if (rc) return rc;
    rc = ensure_tickets(ctx, static_cast<size_t>(B) * Hq, s);
    if (rc) return rc;
    p.part_o = static_cast<float*>(ctx->ws);
    p.part_ml = reinterpret_cast<float2*>(static_cast<char*>(ctx->ws) + o_bytes);
    p.tickets = ctx->tickets;
  }

  dim3 grid(splits, Hq, B);
  cudaError_t e;
  if (a.head_dim == 128) {
    constexpr size_t smem = simt_smem_bytes<128>();
    e = cudaFuncSetAttribute(tree_attn_simt_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaFuncSetAttribute(simt<128>)");
    tree_attn_simt_kernel<128><<<grid, kThreads, smem, s>>>(p);
  } else {
    constexpr size_t smem = simt_smem_bytes<64>();
    e = cudaFuncSetAttribute(tree_attn_simt_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaFuncSetAttribute(simt<64>)");
    tree_attn_simt_kernel<64><<<grid, kThreads, smem, s>>>(p);
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "tree_attn_simt_kernel launch");
  return FALCON_OK;
}

}  // namespace falcon
