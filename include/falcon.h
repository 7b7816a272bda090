/*
 * falcon.h - C ABI of the tree-verification step of Falcon speculative decoding
 * (arXiv 2412.12639) for NVIDIA B200 (sm_100a).
 *
 * One verification step of the target model over the decoding tree is
 *     n_layers x falcon_tree_attn  ->  falcon_tree_accept  ->  falcon_kv_compact
 * (Section 3.4: the drafts form a token tree that the target model verifies in
 * one parallel pass, then "the accepted tokens and their corresponding
 * features" are recorded for the next drafting phase; Section 4.1: greedy
 * decoding, temperature 0).
 *
 * General rules
 *   - Every pointer inside an *_args struct is a DEVICE pointer unless its name
 *     ends in _host.  The structs themselves are host memory and are read
 *     before the call returns.  The caller owns every buffer; the library owns
 *     only the falcon_ctx (scratch memory, cached TMA descriptors).
 *   - `stream` is a cudaStream_t passed as void*.  All work is enqueued on it;
 *     no call synchronises.  A context must not be used from two streams at
 *     the same time (its scratch memory is shared by its calls).
 *   - Return value: FALCON_OK or an error code; on error nothing was launched.
 *   - Faults only the device can see (a malformed parent array, a tree that
 *     does not fit the cache) never trap: the kernel clamps the access, skips
 *     the sequence's result where it must, and ORs FALCON_DEV_* bits into the
 *     optional per-sequence device word tree.status[b].
 *   - A call that needs more scratch memory than the context holds allocates it
 *     (cudaMalloc) and clears what must start at zero on `stream`; make the first
 *     call of each kind and size before capturing the stream into a graph.
 *     Scratch only grows, and a block that was outgrown is kept until
 *     falcon_destroy, so launches already enqueued or captured stay valid.
 *   - There is no CPU fallback and no alternative backend.
 *
 * Tree convention (Section 3.4, Appendix A): a sequence's tree has T <=
 * FALCON_T_MAX single-token nodes with local indices 0..T-1, node 0 is the
 * root (the token the target model has already emitted; a k-token root is a
 * chain of k nodes), parent[0] = -1 and 0 <= parent[i] < i.  Batches are
 * packed: sequence b owns nodes node_off[b] .. node_off[b+1]-1.
 */
#ifndef FALCON_H_
#define FALCON_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FALCON_T_MAX 128

enum {
  FALCON_OK = 0,
  FALCON_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, bad stride          */
  FALCON_ERR_UNSUPPORTED = 2, /* head_dim not 64/128, tree > FALCON_T_MAX, Hq % Hkv   */
  FALCON_ERR_CUDA = 3,        /* a CUDA runtime/driver call failed                    */
  FALCON_ERR_BAD_TREE = 4,    /* host-side tree validation failed                     */
  FALCON_ERR_CAPACITY = 5,    /* sizes exceed a stated maximum                        */
  FALCON_ERR_TIMEOUT = 6      /* a bounded device wait gave up (reported via status)  */
};

/* bits of the optional device status word tree.status[b] */
enum {
  FALCON_DEV_BAD_TREE = 1, /* parent[0] != -1 or parent[i] outside [0, i)            */
  FALCON_DEV_CAPACITY = 2, /* prefix_len + tree size exceeds s_cap                   */
  FALCON_DEV_BAD_PATH = 4, /* path / n_path entry outside the tree (compaction)      */
  FALCON_DEV_TIMEOUT = 8   /* a bounded wait on an on-chip barrier ran out           */
};

typedef struct falcon_ctx falcon_ctx;

/* Creates a context on CUDA device `device` (made current for the call). */
int falcon_create(falcon_ctx** out, int device);
/* Frees the context's scratch memory.  The caller makes sure no work is in flight. */
int falcon_destroy(falcon_ctx* ctx);
/* Static, human-readable name of a return code. */
const char* falcon_status_string(int status);
/* Text of the last CUDA error seen by this context ("" if none). */
const char* falcon_last_error(const falcon_ctx* ctx);
/* Test hook: fills the shared memory and the tensor memory of every SM with `pattern`
 * (0xffffffff is a NaN as bf16 and as fp32), on `stream`.  A kernel launched afterwards that
 * reads on-chip memory it has not written itself then shows it in its results, instead of
 * working by the luck of what an earlier launch left there.  Harmless: plain stores. */
int falcon_test_poison(falcon_ctx* ctx, uint32_t pattern, void* stream);
/* Host check of one tree: FALCON_OK iff T in [1, FALCON_T_MAX], parent[0] == -1
 * and 0 <= parent[i] < i.  `parent` is a HOST pointer. */
int falcon_tree_validate_host(const int32_t* parent, int32_t T);

/* Packed description of the batch of trees shared by the three calls. */
typedef struct {
  int32_t batch;                  /* B >= 1                                             */
  int32_t total_nodes;            /* N = sum of tree sizes (host knows it)              */
  int32_t max_tree;               /* max tree size, <= FALCON_T_MAX                     */
  int32_t max_prefix_len;         /* host upper bound on prefix_len[b] (grid sizing)    */
  const int32_t* node_off;        /* [B+1] node_off[0] = 0                              */
  const int32_t* parent;          /* [N] local parent index, -1 at each local node 0    */
  const int32_t* token;           /* [N] drafted token ids (used by accept only)        */
  const int32_t* prefix_len;      /* [B] rows of the cache that hold the prefix         */
  const int32_t* prefix_len_host; /* optional HOST copy of prefix_len                   */
  const int32_t* node_off_host;   /* optional HOST copy of node_off.  With both host copies (they must
                                     equal the device arrays) small batches skip a device round trip */
  int32_t* status;                /* optional [B] device status words (FALCON_DEV_*)    */
} falcon_tree_desc;

/* ---------------------------------------------------------------------------
 * falcon_tree_attn - tree-masked attention of ONE layer (Section 3.4: the target
 * model scores all tree tokens in one pass with tree attention, each token
 * seeing the prefix and its predecessors in the tree; Section 4.5).
 *
 * For node i of sequence b and query head h (KV head h / (Hq/Hkv)):
 *   keys     {0..L_b-1}  U  {L_b + t : t ancestor-or-self of i}
 *   out[i,h] = softmax_j(sm_scale * q[i,h].K[j]) . V[j]    (fp32 accumulate)
 * tree_mask, when given, replaces "ancestor-or-self" by the set bits of a
 * caller-supplied row (the drafter's relaxed causal mask of Section 3.4).
 *
 * q, out      bf16 [N, Hq, D] contiguous, 16-byte aligned.
 * k/v_cache   bf16, D contiguous, element strides kv_stride_{b,h,s}; row L_b+t
 *             of sequence b holds tree node t's K/V unless k_tree/v_tree given.
 *             Base 16-byte aligned, strides multiples of 8 elements.
 * k/v_tree    optional bf16 [N, Hkv, D]: tree K/V kept outside the cache.
 * kernel      FALCON_ATTN_AUTO picks (by shape, see DESIGN notes in the sources); the others force
 *             one kernel: _SIMT CUDA cores (any supported shape), _WARP CUDA cores with one warp
 *             per query row (at most 1024 keys per sequence; the small-problem kernel), _TC tensor
 *             cores with the query rows on the tensor-memory lanes, _TCK tensor cores with the
 *             keys on the lanes.
 *             The tensor-core kernels need head_dim 128, the tree's K/V in the cache and Hq/Hkv a
 *             power of two; a forced kernel that cannot take the shape returns
 *             FALCON_ERR_UNSUPPORTED.
 * n_splits    0 = automatic; else the number of KV splits per head (1..8 for
 *             the tensor-core kernels, an upper bound: _TCK lowers it when the other
 *             splits' partial results would not fit its shared memory; 1..64 for _SIMT).
 * flags       FALCON_ATTN_PREFIX_STABLE: the caller states that rows [0, L_b) of
 *             k/v_cache were last written by work that had COMPLETED before the
 *             kernel that precedes this call on the stream started (true for a
 *             prefix written in an earlier decoding step).
 *             The tensor-core kernel may then request prefix tiles while that
 *             preceding kernel is still finishing.  Needs the tree's host copies.
 *             Without the flag every read waits for all earlier work of the stream.
 * next_k/v_cache  optional hint for a decoding loop that calls this layer by layer: the
 *             caches the NEXT falcon_tree_attn call on this stream will read, with the same
 *             shape, strides, prefix lengths and FALCON_ATTN_PREFIX_STABLE set.  Once a
 *             thread block has received its own last tile it asks for the next layer's
 *             prefix rows to be brought into L2, so that layer's reads overlap this
 *             layer's tail and the launch gap.  A hint only: results never depend on it,
 *             and only rows [0, L_b) are touched (they must be readable).
 * ------------------------------------------------------------------------- */
enum { FALCON_ATTN_AUTO = 0, FALCON_ATTN_SIMT = 1, FALCON_ATTN_TC = 2, FALCON_ATTN_TCK = 3, FALCON_ATTN_WARP = 4 };
enum {
  FALCON_ATTN_PREFIX_STABLE = 1,
  /* Test hook for the bounded waits of the tensor-core kernels: the first key tile of every thread
   * block is never requested, so the wait for it runs out (about half a second), the kernel sets
   * FALCON_DEV_TIMEOUT in tree.status, drains what is in flight and returns; the context stays
   * usable.  Needs n_splits == 1 and kernel == FALCON_ATTN_TC or _TCK.  The keys-on-lanes kernel still
   * delivers the rows (by its exact fallback path), the other one writes zeros. */
  FALCON_ATTN_TEST_STALL = 1 << 30
};

typedef struct {
  falcon_tree_desc tree;
  int32_t n_q_heads, n_kv_heads, head_dim; /* Hq % Hkv == 0; D in {64, 128}            */
  float sm_scale;                          /* usually 1/sqrt(D)                         */
  const void* q;
  void* out;
  const void* k_cache;
  const void* v_cache;
  int64_t kv_stride_b, kv_stride_h, kv_stride_s;
  int32_t s_cap;                           /* rows per (sequence, head) in the cache    */
  const void* k_tree;
  const void* v_tree;
  const uint64_t* tree_mask;               /* optional [N][2]: bit t of row i = node i sees tree key t */
  int32_t kernel;
  int32_t n_splits;
  int32_t flags;                           /* FALCON_ATTN_* flag bits, 0 = none          */
  const void* next_k_cache;                /* optional hint, see above (NULL = none)     */
  const void* next_v_cache;
} falcon_attn_args;

int falcon_tree_attn(falcon_ctx* ctx, const falcon_attn_args* args, void* stream);
/* Which kernel falcon_tree_attn would run for these arguments (FALCON_ATTN_SIMT, _WARP, _TC or _TCK; for
 * args->kernel == FALCON_ATTN_AUTO the library's choice by shape), or -1 if it would refuse them.
 * Launches nothing; the device pointers are not dereferenced. */
int falcon_tree_attn_kernel(falcon_ctx* ctx, const falcon_attn_args* args);

/* ---------------------------------------------------------------------------
 * falcon_tree_accept - greedy acceptance (Section 4.1 temperature 0; Section 3.4
 * verification as in SpecInfer; the accepted length is tau of Section 4.2).
 *
 *   g[i]      = lowest index of the maximum of logits[i, 0..V-1]  (NaN never wins;
 *               a row with nothing above -inf gives 0)
 *   alive(c)  = every non-root node a on the root..c chain has token[a] == g[parent[a]]
 *   result    = alive node of greatest depth, lowest index among equals
 *   path[b]   = its root-to-node chain (local indices, path[b][0] == 0, rest -1)
 *   n_path[b] = nodes on the path (accepted drafted tokens = n_path - 1)
 *   next_token[b] = g[last node of the path]
 *
 * Non-greedy decoding (temperature > 0).  Section 3.1: the next token is drawn
 * from the distribution that the LM head computes; the paper
 * states no acceptance rule for this case (Appendix A only says the drafted
 * children are sampled; Section 3.4 that verification follows SpecInfer).  The
 * rule here is the simplest one that leaves the output distribution the target's
 * own: at every node the target draws its token and a drafted child is accepted
 * when it carries that token.  The draw is the inverse-CDF one with the caller's
 * uniform number: w_v = exp((logits[i,v] - max) / temperature) (NaN: weight 0),
 * g[i] = lowest v with sum_{k<=v} w_k > uniforms[i] * sum_k w_k (fp32 sums: a
 * draw within rounding of a boundary may fall on either side; a row with no
 * finite maximum gives 0, a +inf logit its first position).  Everything after g
 * is as above.  vocab <= 262144 in this mode.
 * ------------------------------------------------------------------------- */
typedef struct {
  falcon_tree_desc tree;
  int32_t vocab;
  int64_t logits_stride;  /* elements between rows, >= vocab                          */
  const float* logits;    /* fp32 [N, logits_stride]; NULL: g is given, see argmax_out */
  int32_t* argmax_out;    /* [N] g: written; with logits == NULL it is read instead   */
                          /* (e.g. what falcon_lm_head_argmax left there), vocab and  */
                          /* logits_stride are ignored and only the search runs       */
  int32_t* path;          /* [B, path_stride]                                         */
  int32_t path_stride;    /* >= max_tree                                              */
  int32_t* n_path;        /* [B]                                                      */
  int32_t* next_token;    /* [B]                                                      */
  float temperature;      /* 0: greedy, g = the argmax (the paper's setting).  > 0:   */
                          /* non-greedy, g[i] is the target's own draw from           */
                          /* softmax(logits[i] / temperature), see below              */
  const float* uniforms;  /* [N] in [0, 1), one per node; read when temperature > 0   */
} falcon_accept_args;

int falcon_tree_accept(falcon_ctx* ctx, const falcon_accept_args* args, void* stream);

/* ---------------------------------------------------------------------------
 * falcon_lm_head_argmax - the greedy token of every tree node straight from the
 * LM head (Section 3.1: the LM head turns the aggregated features into the
 * distribution over the vocabulary; Eq. 6: p = Softmax(LM(f)); at temperature 0,
 * Section 4.1, only the position of the largest logit matters).  The [N, vocab]
 * logits are never written to memory:
 *
 *   logit[i, v]   = sum_k features[i, k] * lm_head[v, k]     (bf16 inputs, fp32 sums)
 *   argmax_out[i] = lowest v attaining the maximum (NaN never wins; a row with
 *                   nothing above -inf gives 0)
 *   max_out[i]    = that logit (optional)
 *
 * The head is a bias-free linear map stored row by row ([vocab, hidden], what the
 * LLaMA / Vicuna checkpoints hold) and a constant: the kernel starts reading it
 * while the previous kernel of the stream is still finishing, so that kernel must
 * not be the one that writes lm_head.  falcon_tree_accept with logits == NULL then
 * finds the accepted path from argmax_out.  The sums are taken in fp32 in the
 * tensor core's order: two logits closer than that rounding may swap places
 * relative to an exact evaluation.
 *   limits   n_rows <= 65535; both pitches multiples of 8 elements and both bases
 *            16-byte aligned (FALCON_ERR_UNSUPPORTED otherwise)
 *   status   optional device word; FALCON_DEV_TIMEOUT is set there if a bounded
 *            wait inside the kernel gave up (the results are then not valid)
 * Device pointers; the caller owns every buffer; scratch comes from the context.
 * ------------------------------------------------------------------------- */
/* Test hook: the features of the first pipeline stage are never requested, so the kernel's first
 * bounded wait runs out: FALCON_DEV_TIMEOUT in *status, the kernel returns in order, the context
 * stays usable.  (No fault, no hang: every wait in the kernel has a limit.) */
#define FALCON_LM_TEST_STALL (1 << 30)
typedef struct {
  int32_t n_rows;         /* N: rows of `features` (tree nodes)                        */
  int32_t hidden;
  int32_t vocab;
  const void* features;   /* bf16 [n_rows, feat_stride]                                */
  int64_t feat_stride;    /* elements between rows, >= hidden                          */
  const void* lm_head;    /* bf16 [vocab, head_stride]                                 */
  int64_t head_stride;    /* elements between rows, >= hidden                          */
  int32_t* argmax_out;    /* [n_rows]                                                  */
  float* max_out;         /* [n_rows] or NULL                                          */
  int32_t* status;        /* 1 word or NULL                                            */
  int32_t flags;          /* 0, or FALCON_LM_TEST_STALL                                */
} falcon_lm_argmax_args;

int falcon_lm_head_argmax(falcon_ctx* ctx, const falcon_lm_argmax_args* args, void* stream);

/* ---------------------------------------------------------------------------
 * falcon_topm - the m best entries of every logits row, best first: the children
 * a node of the decoding tree is given when the tree is grown (Appendix A: in the
 * greedy setting the m most probable tokens, m = 20 at the root).  It is the step just
 * before verification and scans the same kind of [rows, vocab] fp32 matrix as
 * the acceptance call.
 *
 *   order      larger value first; the lower index among equal values (+0 == -0);
 *              a NaN counts as -inf and is reported as -inf
 *   top_val    [n_rows, m] fp32, top_idx [n_rows, m] int32, row-major, device memory
 *   limits     1 <= m <= min(vocab, FALCON_TOPM_MAX); vocab <= 262144;
 *              n_rows <= 65535; logits 4-byte aligned
 * Errors: FALCON_ERR_INVALID_ARG / FALCON_ERR_CAPACITY, nothing launched.  Scratch
 * comes from the context (the first call of a size allocates it).
 * ------------------------------------------------------------------------- */
#define FALCON_TOPM_MAX 32
typedef struct {
  int32_t n_rows;
  int32_t vocab;
  int64_t logits_stride;  /* elements between rows, >= vocab                          */
  const float* logits;    /* fp32 [n_rows, logits_stride]                             */
  int32_t m;
  float* top_val;         /* [n_rows, m]                                              */
  int32_t* top_idx;       /* [n_rows, m]                                              */
} falcon_topm_args;

int falcon_topm(falcon_ctx* ctx, const falcon_topm_args* args, void* stream);

/* ---------------------------------------------------------------------------
 * falcon_tree_accept_static - falcon_tree_accept for callers that cannot allocate
 * device memory.  (The paper has no counterpart: this is a deployment variant of
 * the call above, same arguments, same results.)
 *
 * Who needs it: a serving process whose device memory is owned entirely by its
 * own pool, a process pinned to a fixed memory budget, or a latency-critical
 * loop that cannot risk the device-wide synchronisation an allocation can cause.
 * This call needs no falcon_ctx and never calls cudaMalloc, cudaFree or any
 * allocating routine.  Its scratch (argmax partials, arrival counters) is a fixed
 * array inside the library image, about 0.5 MB, which every GPU that loads the
 * library holds until the process exits.
 *
 * Limits: total_nodes <= FALCON_STATIC_MAX_NODES and batch <=
 * FALCON_STATIC_MAX_BATCH; anything larger returns FALCON_ERR_CAPACITY and
 * launches nothing.  It runs on the current device, and `stream` must be a stream
 * of that device (the array's address differs from device to device).  The first call on each
 * device looks up the array's device address (a one-time set-up step); make that
 * first call before any stream capture begins.  All calls on a device share the
 * one array, and it keeps the previous call's contents: the call itself clears
 * the counters it needs at zero, but two calls that overlap on the GPU (different
 * streams, no ordering between them) race on it and give wrong results -
 * serialise them.
 * ------------------------------------------------------------------------- */
#define FALCON_STATIC_MAX_NODES 1024
#define FALCON_STATIC_MAX_BATCH 256
int falcon_tree_accept_static(const falcon_accept_args* args, void* stream);

/* ---------------------------------------------------------------------------
 * falcon_feature_gather - the accepted tokens and their features (Section 3.4: after
 * verification they are kept for the next drafting phase: the drafter's next input is the
 * target model's hidden state of every accepted node together with its token, Section 3.1).
 *
 *   tokens_out[b, j]      = token[node_off[b] + path[b][j]]
 *   features_out[b, j, :] = features[node_off[b] + path[b][j], 0 .. hidden-1]    j < n_path[b]
 * Rows j >= n_path[b] of the outputs are not written.  Features are 16-bit elements
 * (bf16), copied bit for bit.  A path entry outside the tree sets FALCON_DEV_BAD_PATH
 * and leaves that sequence's outputs alone.
 *
 *   features      [N, feat_stride], feat_stride >= hidden, both multiples of 8, 16-byte aligned
 *   features_out  [B, out_rows, hidden], tokens_out [B, out_rows], out_rows >= max_tree
 * The same work can ride on the compaction launch: see falcon_compact_args.gather.
 * ------------------------------------------------------------------------- */
typedef struct {
  falcon_tree_desc tree;  /* token is read                                            */
  int32_t hidden;
  int64_t feat_stride;
  const void* features;
  const int32_t* path;    /* [B, path_stride] from falcon_tree_accept                 */
  int32_t path_stride;
  const int32_t* n_path;  /* [B]                                                      */
  int32_t out_rows;
  void* features_out;
  int32_t* tokens_out;
} falcon_gather_args;

int falcon_feature_gather(falcon_ctx* ctx, const falcon_gather_args* args, void* stream);

/* ---------------------------------------------------------------------------
 * falcon_kv_compact - keep the accepted path's K/V (Section 3.4: the accepted tokens
 * and their features are kept for the next drafting phase; this is the KV-cache form
 * of that step), all layers in one launch.
 *
 *   cache row L_b + j  <-  tree row path[b][j],   j = 0 .. n_path[b]-1
 *   new_len[b] = L_b + n_path[b]
 * In place by default (tree row t is cache row L_b + t; a destination row may be
 * an earlier source row, which the kernel handles); with k/v_tree_layers the tree
 * rows come from separate [N, Hkv, D] buffers.  Rows below L_b are untouched;
 * rows at and above new_len[b] are unspecified afterwards.  prefix_len is not
 * modified.
 * ------------------------------------------------------------------------- */
typedef struct {
  falcon_tree_desc tree;  /* token unused (read only when `gather` is given)          */
  int32_t n_layers, n_kv_heads, head_dim;
  void* const* k_cache_layers; /* device array [n_layers] of cache base pointers      */
  void* const* v_cache_layers;
  int64_t kv_stride_b, kv_stride_h, kv_stride_s;
  int32_t s_cap;
  const void* const* k_tree_layers; /* optional device array [n_layers]               */
  const void* const* v_tree_layers;
  const int32_t* path;    /* [B, path_stride] from falcon_tree_accept                 */
  int32_t path_stride;
  const int32_t* n_path;  /* [B]                                                      */
  int32_t* new_len;       /* [B]                                                      */
  const falcon_gather_args* gather; /* optional HOST pointer: also record the accepted tokens and features in
                                       this launch (its features / outputs are used; tree, path and n_path
                                       are the compaction's, which must describe the same batch)         */
} falcon_compact_args;

int falcon_kv_compact(falcon_ctx* ctx, const falcon_compact_args* args, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* FALCON_H_ */
