"""GPU parity: the CUDA library, called through the C ABI, against the CPU oracle
on the same seeded inputs.  Integer outputs and caches are compared bit for bit;
attention within max-abs 2e-2 and per-(sequence, head) relative L2 1e-2."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2412_12639_b200 import binding, synth

import gpu_harness as H

pytestmark = pytest.mark.gpu

KERNELS = [binding.ATTN_SIMT, binding.ATTN_WARP, binding.ATTN_TC, binding.ATTN_TCK]
TC_KERNELS = [binding.ATTN_TC, binding.ATTN_TCK]      # queries / keys on the tensor-memory lanes


def tc_or_skip(rc):
    if rc == binding.ERR_UNSUPPORTED:
        pytest.skip("shape not taken by this kernel")
    assert rc == binding.OK


def strides_of(a):
    return tuple(s // 2 for s in a.strides[:3])


def oracle_attn(tb, Hq, Hkv, D, q, k, v, scale=None, **kw):
    scale = 1.0 / math.sqrt(D) if scale is None else scale
    return oracle.tree_attn(tb.node_off, tb.parent, tb.prefix_len, Hq, Hkv, D, scale, q, k, v, strides_of(k), **kw)


def random_case(rng, sizes, prefs, Hq, Hkv, D, slack=0):
    tb = H.make_trees(sizes, prefs, rng)
    s_cap = int(max(p + t for p, t in zip(prefs, sizes))) + slack
    q = synth.normal_bf16(rng, (tb.total_nodes, Hq, D))
    k = synth.normal_bf16(rng, (tb.batch, Hkv, s_cap, D))
    v = synth.normal_bf16(rng, (tb.batch, Hkv, s_cap, D))
    return tb, q, k, v


# ------------------------------------------------------------------ attention
@pytest.mark.parametrize("kernel", KERNELS)
def test_attn_tiny_config(kernel):
    spec = synth.SPECS["tiny"]
    tb = synth.make_trees(spec)
    q, k, v = synth.make_layer_qkv(spec, tb, 0)
    ref = oracle_attn(tb, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, q, k, v)
    out, rc = H.run_attn(H.DevTrees(tb), spec.n_q_heads, spec.n_kv_heads, spec.head_dim, q, k, v, kernel=kernel,
                         check=False)
    tc_or_skip(rc)
    H.assert_attn_close(out, ref, tb.node_off)


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("G", [1, 2, 4, 8])
def test_attn_sweep_shapes(kernel, D, G):
    rng = np.random.default_rng(1000 * D + G)
    Hkv = 2
    for T, L in [(1, 0), (1, 1), (2, 31), (15, 32), (33, 33), (60, 127), (64, 128), (65, 129), (128, 200),
                 (97, 333), (128, 0)]:
        tb, q, k, v = random_case(rng, [T], [L], Hkv * G, Hkv, D, slack=int(rng.integers(0, 5)))
        ref = oracle_attn(tb, Hkv * G, Hkv, D, q, k, v)
        out, rc = H.run_attn(H.DevTrees(tb), Hkv * G, Hkv, D, q, k, v, kernel=kernel, check=False)
        tc_or_skip(rc)
        H.assert_attn_close(out, ref, tb.node_off)


@pytest.mark.parametrize("kernel", KERNELS)
def test_attn_split_invariance_and_determinism(kernel):
    rng = np.random.default_rng(7)
    tb, q, k, v = random_case(rng, [60], [1024], 4, 4, 128)
    ref = oracle_attn(tb, 4, 4, 128, q, k, v)
    dt = H.DevTrees(tb)
    outs = []
    for splits in (1, 2, 3, 8):
        out, rc = H.run_attn(dt, 4, 4, 128, q, k, v, kernel=kernel, n_splits=splits, check=False)
        tc_or_skip(rc)
        H.assert_attn_close(out, ref, tb.node_off)
        out2, _ = H.run_attn(dt, 4, 4, 128, q, k, v, kernel=kernel, n_splits=splits)
        np.testing.assert_array_equal(out, out2)       # same launch twice: bit-identical
        outs.append(out)


@pytest.mark.parametrize("kernel", KERNELS)
def test_attn_host_copies_of_the_scalars_change_nothing(kernel):
    rng = np.random.default_rng(22)
    for sizes, prefs in (([60], [1024]), ([20, 80, 33], [300, 40, 129]), ([7] * 9, [65] * 9)):   # 9 > host table size
        tb, q, k, v = random_case(rng, sizes, prefs, 4, 2, 128, slack=2)
        ref = oracle_attn(tb, 4, 2, 128, q, k, v)
        dt = H.DevTrees(tb)
        a, rc = H.run_attn(dt, 4, 2, 128, q, k, v, kernel=kernel, check=False)
        tc_or_skip(rc)
        b, _ = H.run_attn(dt, 4, 2, 128, q, k, v, kernel=kernel, host_copies=True)
        np.testing.assert_array_equal(a, b)
        H.assert_attn_close(b, ref, tb.node_off)


@pytest.mark.parametrize("kernel", KERNELS)
def test_attn_ragged_batch_small(kernel):
    rng = np.random.default_rng(21)
    sizes = [20, 80, 1, 47, 64, 33]
    prefs = [256, 40, 700, 0, 513, 129]
    tb, q, k, v = random_case(rng, sizes, prefs, 4, 2, 128, slack=3)
    ref = oracle_attn(tb, 4, 2, 128, q, k, v)
    out, rc = H.run_attn(H.DevTrees(tb), 4, 2, 128, q, k, v, kernel=kernel, check=False)
    tc_or_skip(rc)
    H.assert_attn_close(out, ref, tb.node_off)


@pytest.mark.parametrize("kernel", KERNELS)
def test_attn_chain_star_and_wide_root(kernel):
    rng = np.random.default_rng(5)
    for parent in (synth.chain_tree(40), synth.star_tree(21), synth.chain_tree(128), synth.star_tree(128)):
        T = len(parent)
        tb = H.make_trees([T], [77], rng, parents=[parent])
        q = synth.normal_bf16(rng, (T, 2, 128))
        k = synth.normal_bf16(rng, (1, 2, 77 + T, 128))
        v = synth.normal_bf16(rng, (1, 2, 77 + T, 128))
        ref = oracle_attn(tb, 2, 2, 128, q, k, v)
        out, rc = H.run_attn(H.DevTrees(tb), 2, 2, 128, q, k, v, kernel=kernel, check=False)
        tc_or_skip(rc)
        H.assert_attn_close(out, ref, tb.node_off)


@pytest.mark.parametrize("kernel", KERNELS)
def test_attn_ignores_rows_past_the_tree_even_if_nan(kernel):
    rng = np.random.default_rng(6)
    tb, q, k, v = random_case(rng, [30, 17], [100, 60], 2, 2, 128, slack=40)
    for b in range(2):
        end = tb.prefix_len[b] + tb.tree_size(b)
        k[b, :, end:] = 0x7FC0      # NaN
        v[b, :, end:] = 0x7F80      # +inf
    ref = oracle_attn(tb, 2, 2, 128, q, k, v)
    out, rc = H.run_attn(H.DevTrees(tb), 2, 2, 128, q, k, v, kernel=kernel, check=False)
    tc_or_skip(rc)
    H.assert_attn_close(out, ref, tb.node_off)


@pytest.mark.parametrize("kernel", KERNELS)
def test_attn_large_scores_do_not_overflow(kernel):
    # keys whose scores grow along the sequence, with a big scale: the running maximum keeps moving up
    rng = np.random.default_rng(8)
    T, L, D = 24, 300, 128
    tb = H.make_trees([T], [L], rng)
    q = synth.f32_to_bf16_bits(np.ones((T, 1, D), np.float32))
    ramp = np.linspace(-2.0, 2.0, L + T, dtype=np.float32)[None, None, :, None]
    k = synth.f32_to_bf16_bits(np.broadcast_to(ramp, (1, 1, L + T, D)).copy())
    v = synth.normal_bf16(rng, (1, 1, L + T, D))
    ref = oracle_attn(tb, 1, 1, D, q, k, v, scale=1.0)
    out, rc = H.run_attn(H.DevTrees(tb), 1, 1, D, q, k, v, scale=1.0, kernel=kernel, check=False)
    tc_or_skip(rc)
    H.assert_attn_close(out, ref, tb.node_off)


@pytest.mark.parametrize("kernel", KERNELS)
def test_attn_separate_tree_buffers(kernel):
    rng = np.random.default_rng(9)
    sizes, prefs = [40, 9], [130, 0]
    tb, q, k, v = random_case(rng, sizes, prefs, 4, 2, 128)
    kt = np.empty((tb.total_nodes, 2, 128), np.uint16)
    vt = np.empty_like(kt)
    k2, v2 = k.copy(), v.copy()
    for b in range(2):
        L, T, o = prefs[b], sizes[b], tb.node_off[b]
        kt[o:o + T] = k[b, :, L:L + T].transpose(1, 0, 2)
        vt[o:o + T] = v[b, :, L:L + T].transpose(1, 0, 2)
        k2[b, :, L:] = 0x7FC0
        v2[b, :, L:] = 0x7FC0
    ref = oracle_attn(tb, 4, 2, 128, q, k, v)
    out, rc = H.run_attn(H.DevTrees(tb), 4, 2, 128, q, k2, v2, k_tree=kt, v_tree=vt, kernel=kernel, check=False)
    tc_or_skip(rc)
    H.assert_attn_close(out, ref, tb.node_off)


def relaxed_mask_rows(tb, k_block, drop=()):
    """Mask rows of the drafter's relaxed causal mask (Section 3.4): a node sees its predecessors in the tree and the
    nodes of its own block of k_block consecutive nodes.  `drop` lists (packed node, tree key) bits to clear."""
    rows = np.zeros((tb.total_nodes, 2), np.uint64)
    for b in range(tb.batch):
        o, T = int(tb.node_off[b]), tb.tree_size(b)
        par = tb.parent[o:o + T]
        for i in range(T):
            vis = set(oracle.ancestors(par, i)) | {m for m in range(i - i % k_block, min(T, i - i % k_block + k_block))}
            for a in vis:
                rows[o + i, a >> 6] |= np.uint64(1) << np.uint64(a & 63)
    for node, key in drop:
        rows[node, key >> 6] &= ~(np.uint64(1) << np.uint64(key & 63))
    return rows


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("splits", [0, 3])
def test_attn_caller_mask_rows(kernel, splits):
    # relaxed causal mask of the drafter on a batch of two sequences with different tree sizes and prefixes, one row
    # with an ancestor bit cleared: the rows of the second sequence start at a non-zero packed offset
    rng = np.random.default_rng(10)
    sizes, prefs = [50, 77], [90, 301]
    tb, q, k, v = random_case(rng, sizes, prefs, 4, 2, 128, slack=2)
    rows = relaxed_mask_rows(tb, 3, drop=[(50 + 40, int(tb.parent[50 + 40]))])
    ref = oracle_attn(tb, 4, 2, 128, q, k, v, tree_mask=rows)
    plain = oracle_attn(tb, 4, 2, 128, q, k, v)
    assert np.abs(ref - plain).max() > 0.05            # the mask rows do change the result
    out, rc = H.run_attn(H.DevTrees(tb), 4, 2, 128, q, k, v, tree_mask=rows, kernel=kernel, n_splits=splits, check=False)
    tc_or_skip(rc)
    H.assert_attn_close(out, ref, tb.node_off)


@pytest.mark.parametrize("kernel", KERNELS)
def test_attn_strided_cache_view(kernel):
    # K and V interleaved in one allocation: [B, Hkv, s_cap, 2, D] -> row stride 2*D
    rng = np.random.default_rng(12)
    T, L, D = 33, 140, 128
    tb = H.make_trees([T], [L], rng)
    q = synth.normal_bf16(rng, (T, 2, D))
    kv = synth.normal_bf16(rng, (1, 2, L + T, 2, D))
    k, v = kv[:, :, :, 0], kv[:, :, :, 1]
    ref = oracle.tree_attn(tb.node_off, tb.parent, tb.prefix_len, 2, 2, D, 1 / math.sqrt(D), q, k, v, strides_of(k))
    kvd = H.dev_bf16(kv)
    qd = H.dev_bf16(q)
    out = torch.zeros_like(qd)
    dt = H.DevTrees(tb)
    kd, vd = kvd[:, :, :, 0], kvd[:, :, :, 1]
    a = binding.attn_args(dt.desc(), 2, 2, D, 1 / math.sqrt(D), qd, out, kd.data_ptr(), vd.data_ptr(),
                          tuple(int(s) for s in kd.stride()[:3]), L + T, kernel=kernel)
    rc = H.ctx().falcon_tree_attn(a, check=False)
    tc_or_skip(rc)
    torch.cuda.synchronize()
    H.assert_attn_close(H.host_bits(out), ref, tb.node_off)


def test_attn_malformed_tree_and_capacity_set_status_without_faulting():
    rng = np.random.default_rng(13)
    tb, q, k, v = random_case(rng, [10, 12], [20, 30], 2, 2, 128)
    tb.parent[3] = 7                      # parent after child in sequence 0
    dt = H.DevTrees(tb)
    for kernel in KERNELS:
        dt.status.zero_()
        out, rc = H.run_attn(dt, 2, 2, 128, q, k, v, kernel=kernel, check=False)
        if rc == binding.ERR_UNSUPPORTED:
            continue
        st = dt.status.cpu().numpy()
        assert st[0] & binding.DEV_BAD_TREE and st[1] == 0
        # sequence 1 is well formed: its rows are still right
        ref = oracle_attn(synth.TreeBatch(np.array([0, 12], np.int32), tb.parent[10:], tb.token[10:],
                                          tb.prefix_len[1:], tb.p_accept[1:]), 2, 2, 128, q[10:], k[1:], v[1:])
        H.assert_attn_close(out[10:], ref, np.array([0, 12]))
    # tree rows that do not fit the cache
    tb2, q, k, v = random_case(rng, [10], [20], 2, 2, 128)
    dt2 = H.DevTrees(tb2)
    for kernel in KERNELS:
        dt2.status.zero_()
        _, rc = H.run_attn(dt2, 2, 2, 128, q, k, v, s_cap=25, kernel=kernel, check=False)
        if rc == binding.ERR_UNSUPPORTED:
            continue
        assert dt2.status.cpu().numpy()[0] & binding.DEV_CAPACITY


FULL = {"v7b": list(range(32)), "l13b": list(range(40)), "l70b": [1, 5], "ragged": [2, 30]}   # KV heads the oracle checks


@pytest.mark.parametrize("name", ["v7b", "l13b", "l70b", "ragged"])
def test_attn_full_size_configs_sampled_heads(name):
    """Full-size launch (the one the benchmark times); the oracle checks every head of one layer of the two graded
    shapes and a sample of KV heads of the two large ones, per (node, head) row."""
    spec = synth.SPECS[name]
    tb = synth.make_trees(spec)
    q, k, v = synth.make_layer_qkv(spec, tb, 1)
    # as the benchmark launches it: host copies of the scalars, stable prefix
    out, _ = H.run_attn(H.DevTrees(tb), spec.n_q_heads, spec.n_kv_heads, spec.head_dim, q, k, v, host_copies=True,
                        flags=binding.ATTN_PREFIX_STABLE)
    G = spec.n_q_heads // spec.n_kv_heads
    for kvh in [h % spec.n_kv_heads for h in FULL[name]]:
        qs = np.ascontiguousarray(q[:, kvh * G:(kvh + 1) * G])
        ks = np.ascontiguousarray(k[:, kvh:kvh + 1])
        vs = np.ascontiguousarray(v[:, kvh:kvh + 1])
        ref = oracle_attn(tb, G, 1, spec.head_dim, qs, ks, vs)
        H.assert_attn_close(np.ascontiguousarray(out[:, kvh * G:(kvh + 1) * G]), ref, tb.node_off, report=kvh == FULL[name][0])


# --------------------------------------------------------------------- accept
@pytest.mark.parametrize("name", ["tiny", "v7b", "l13b", "l70b", "ragged"])
def test_accept_configs_bit_exact(name):
    spec = synth.SPECS[name]
    tb = synth.make_trees(spec)
    logits = synth.make_logits(spec, tb)
    g_ref = oracle.argmax(logits)
    p_ref, n_ref, t_ref = oracle.tree_accept(tb.node_off, tb.parent, tb.token, g_ref)
    g, path, n, nxt = H.run_accept(H.DevTrees(tb), logits)
    np.testing.assert_array_equal(g, g_ref)
    np.testing.assert_array_equal(n, n_ref)
    np.testing.assert_array_equal(path, p_ref)
    np.testing.assert_array_equal(nxt, t_ref)
    # a second call on the same context gives the same result (arrival counters were reset)
    g2, path2, n2, nxt2 = H.run_accept(H.DevTrees(tb), logits)
    np.testing.assert_array_equal(path2, p_ref)
    np.testing.assert_array_equal(g2, g_ref)


@pytest.mark.parametrize("V,stride", [(1, 1), (3, 5), (1000, 1000), (4099, 4101), (32001, 32001), (32000, 32004),
                                      (50000, 50001)])
def test_accept_argmax_odd_vocab_and_strides(V, stride):
    rng = np.random.default_rng(V)
    tb = H.make_trees([37, 5], [0, 0], rng, vocab=max(1, min(V, 50)))
    logits = rng.standard_normal((42, stride)).astype(np.float32)
    logits[:, V:] = 100.0                              # padding columns must be ignored
    g_ref = oracle.argmax(logits, vocab=V)
    p_ref, n_ref, t_ref = oracle.tree_accept(tb.node_off, tb.parent, tb.token, g_ref)
    g, path, n, nxt = H.run_accept(H.DevTrees(tb), logits, vocab=V)
    np.testing.assert_array_equal(g, g_ref)
    np.testing.assert_array_equal(path, p_ref)
    np.testing.assert_array_equal(n, n_ref)
    np.testing.assert_array_equal(nxt, t_ref)


def test_accept_argmax_ties_nan_inf_and_signed_zero():
    rng = np.random.default_rng(3)
    V = 9000
    tb = H.make_trees([8], [0], rng)
    x = rng.standard_normal((8, V)).astype(np.float32)
    x[0, [100, 5000, 8999]] = 77.0                     # ties far apart (different chunks): lowest index
    x[1] = np.nan
    x[2] = -np.inf
    x[3] = 0.0
    x[3, ::2] = -0.0
    x[4, :4000] = np.nan
    x[4, 4000:] = -np.inf                              # nothing above -inf: 0
    x[5, 17] = np.inf
    x[5, 16] = np.nan
    x[6, :] = -np.inf
    x[6, 8191] = -3.0
    x[7, 0] = np.nan
    x[7, 1:] = -np.inf
    g_ref = oracle.argmax(x)
    assert g_ref.tolist()[:8] == [100, 0, 0, 0, 0, 17, 8191, 0]
    g, _, _, _ = H.run_accept(H.DevTrees(tb), x)
    np.testing.assert_array_equal(g, g_ref)


@pytest.mark.parametrize("seed", range(4))
def test_accept_random_trees_small_vocab_bit_exact(seed):
    rng = np.random.default_rng(seed)
    sizes = [int(rng.integers(1, 129)) for _ in range(16)]
    tb = H.make_trees(sizes, [0] * 16, rng, vocab=5)
    logits = rng.standard_normal((tb.total_nodes, 5)).astype(np.float32)
    g_ref = oracle.argmax(logits)
    p_ref, n_ref, t_ref = oracle.tree_accept(tb.node_off, tb.parent, tb.token, g_ref)
    g, path, n, nxt = H.run_accept(H.DevTrees(tb), logits)
    np.testing.assert_array_equal(g, g_ref)
    np.testing.assert_array_equal(path, p_ref)
    np.testing.assert_array_equal(n, n_ref)
    np.testing.assert_array_equal(nxt, t_ref)


def test_accept_malformed_tree_reports_and_returns_root():
    rng = np.random.default_rng(2)
    tb = H.make_trees([6, 6], [0, 0], rng, vocab=4)
    tb.parent[8] = 5                                   # sequence 1: parent[2] = 5 >= 2
    logits = rng.standard_normal((12, 4)).astype(np.float32)
    dt = H.DevTrees(tb)
    g, path, n, nxt = H.run_accept(dt, logits)
    st = dt.status.cpu().numpy()
    assert st[0] == 0 and st[1] & binding.DEV_BAD_TREE
    assert n[1] == 1 and path[1, 0] == 0 and nxt[1] == g[6]


# -------------------------------------------------------------------- compact
def accepted_paths(tb, rng, force=None):
    B = tb.batch
    path = np.full((B, 128), -1, np.int32)
    n_path = np.zeros(B, np.int32)
    for b in range(B):
        par = tb.parent[tb.node_off[b]:tb.node_off[b + 1]]
        node = int(rng.integers(0, len(par))) if force is None else force[b]
        chain = oracle.ancestors(par, node)[::-1]
        path[b, :len(chain)] = chain
        n_path[b] = len(chain)
    return path, n_path


def check_compact(tb, Hkv, D, n_layers, rng, path, n_path, separate=False, slack=2):
    s_cap = int((tb.prefix_len + np.diff(tb.node_off)).max()) + slack
    ks = [rng.integers(0, 65536, size=(tb.batch, Hkv, s_cap, D)).astype(np.uint16) for _ in range(n_layers)]
    vs = [rng.integers(0, 65536, size=(tb.batch, Hkv, s_cap, D)).astype(np.uint16) for _ in range(n_layers)]
    kt = vt = None
    if separate:
        kt = [rng.integers(0, 65536, size=(tb.total_nodes, Hkv, D)).astype(np.uint16) for _ in range(n_layers)]
        vt = [rng.integers(0, 65536, size=(tb.total_nodes, Hkv, D)).astype(np.uint16) for _ in range(n_layers)]
    gk, gv, new_len = H.run_compact(H.DevTrees(tb), Hkv, D, ks, vs, path, n_path, kt, vt)
    for l in range(n_layers):
        for ref, got, tree in ((ks[l], gk[l], kt), (vs[l], gv[l], vt)):
            before = ref.copy()
            nl = oracle.kv_compact(tb.node_off, tb.prefix_len, Hkv, D, ref, strides_of(ref), s_cap, path, n_path,
                                   tree_rows=None if tree is None else (kt[l] if ref is ks[l] else vt[l]))
            np.testing.assert_array_equal(new_len, nl)
            for b in range(tb.batch):
                np.testing.assert_array_equal(got[b, :, :nl[b]], ref[b, :, :nl[b]])
                np.testing.assert_array_equal(got[b, :, :tb.prefix_len[b]], before[b, :, :tb.prefix_len[b]])


@pytest.mark.parametrize("name,layers", [("tiny", 1), ("v7b", 3), ("l13b", 2), ("l70b", 3), ("ragged", 2)])
def test_compact_configs_bit_exact_with_accepted_paths(name, layers):
    spec = synth.SPECS[name]
    tb = synth.make_trees(spec)
    logits = synth.make_logits(spec, tb)
    g = oracle.argmax(logits)
    path, n_path, _ = oracle.tree_accept(tb.node_off, tb.parent, tb.token, g)
    check_compact(tb, spec.n_kv_heads, spec.head_dim, layers, np.random.default_rng(0), path, n_path)


@pytest.mark.parametrize("separate", [False, True])
@pytest.mark.parametrize("D", [64, 128, 256])
def test_compact_random_paths_overlap_and_identity(separate, D):
    rng = np.random.default_rng(D + separate)
    sizes = [128, 1, 40, 77]
    parents = [synth.chain_tree(128), np.array([-1], np.int32), synth.random_shape_tree(rng, 40),
               synth.random_shape_tree(rng, 77)]
    tb = H.make_trees(sizes, [5, 0, 64, 300], rng, parents=parents)
    # full chain of 128 (identity, the largest copy), single node, two random leaves
    path, n_path = accepted_paths(tb, rng, force=[127, 0, 39, 76])
    check_compact(tb, 3, D, 2, rng, path, n_path, separate=separate)
    path, n_path = accepted_paths(tb, rng)
    check_compact(tb, 3, D, 2, rng, path, n_path, separate=separate)


def test_compact_handworked_overlap_path():
    rng = np.random.default_rng(4)
    tb = H.make_trees([4], [2], rng, parents=[np.array([-1, 0, 0, 2], np.int32)])
    path = np.full((1, 128), -1, np.int32)
    path[0, :3] = [0, 2, 3]
    check_compact(tb, 2, 64, 1, rng, path, np.array([3], np.int32), slack=0)


def test_compact_bad_path_or_capacity_leaves_cache_untouched():
    rng = np.random.default_rng(5)
    tb = H.make_trees([6, 6], [4, 4], rng)
    path = np.full((2, 128), -1, np.int32)
    path[:, 0] = 0
    path[1, 1] = 9                                      # outside the tree
    n_path = np.array([1, 2], np.int32)
    s_cap = 12
    ks = [rng.integers(0, 65536, size=(2, 2, s_cap, 64)).astype(np.uint16)]
    vs = [rng.integers(0, 65536, size=(2, 2, s_cap, 64)).astype(np.uint16)]
    dt = H.DevTrees(tb)
    gk, gv, new_len = H.run_compact(dt, 2, 64, ks, vs, path, n_path)
    st = dt.status.cpu().numpy()
    assert st[0] == 0 and st[1] & binding.DEV_BAD_PATH
    assert new_len.tolist() == [5, 4]
    np.testing.assert_array_equal(gk[0][1], ks[0][1])
    np.testing.assert_array_equal(gv[0][1], vs[0][1])


def test_compact_path_longer_than_the_declared_max_tree_is_refused():
    """The launcher picks the copy variant from the caller's max_tree; a sequence whose path does not
    fit that variant is reported (capacity) and its cache is left alone, the other sequence is compacted."""
    rng = np.random.default_rng(6)
    tb = H.make_trees([100, 8], [10, 3], rng, parents=[synth.chain_tree(100), synth.chain_tree(8)])
    path = np.full((2, 128), -1, np.int32)
    path[0, :80] = np.arange(80)                       # 80 rows x 16 chunks = 1280 > 1024: too long for the small variant
    path[1, :5] = np.arange(5)
    n_path = np.array([80, 5], np.int32)
    s_cap = 112
    ks = [rng.integers(0, 65536, size=(2, 2, s_cap, 128)).astype(np.uint16)]
    vs = [rng.integers(0, 65536, size=(2, 2, s_cap, 128)).astype(np.uint16)]
    dt = H.DevTrees(tb)
    honest = dt.desc

    def understated(**kw):
        d = honest(**kw)
        d.max_tree = 60                                 # passes the host check (60 x 2 >= 108 nodes), still too small
        return d

    dt.desc = understated
    gk, gv, new_len = H.run_compact(dt, 2, 128, ks, vs, path, n_path)
    st = dt.status.cpu().numpy()
    assert st[0] & binding.DEV_CAPACITY and st[1] == 0
    assert new_len.tolist() == [10, 8]
    np.testing.assert_array_equal(gk[0][0], ks[0][0])
    np.testing.assert_array_equal(gv[0][0], vs[0][0])
    ref_k, ref_v = ks[0].copy(), vs[0].copy()
    for ref in (ref_k, ref_v):
        oracle.kv_compact(tb.node_off, tb.prefix_len, 2, 128, ref, strides_of(ref), s_cap, path, n_path)
    np.testing.assert_array_equal(gk[0][1, :, :8], ref_k[1, :, :8])
    np.testing.assert_array_equal(gv[0][1, :, :8], ref_v[1, :, :8])


@pytest.mark.parametrize("tck", TC_KERNELS)
@pytest.mark.parametrize("T,G,L,splits", [(60, 1, 700, 1), (60, 1, 700, 4), (32, 2, 100, 2), (17, 1, 0, 1),
                                           (80, 1, 30, 2), (80, 1, 500, 1), (128, 1, 64, 3), (16, 8, 1000, 5)])
def test_attn_tc_row_arrangements(T, G, L, splits, tck):
    """Both arrangements of the tensor-core kernel (two copies of at most 64 rows; two streams on
    alternate tiles, including runs of a single tile where the second stream has nothing) at forced splits."""
    rng = np.random.default_rng(100 * T + 10 * G + splits)
    Hkv = 2
    tb, q, k, v = random_case(rng, [T], [L], Hkv * G, Hkv, 128, slack=1)
    ref = oracle_attn(tb, Hkv * G, Hkv, 128, q, k, v)
    out, rc = H.run_attn(H.DevTrees(tb), Hkv * G, Hkv, 128, q, k, v, kernel=tck, n_splits=splits,
                         check=False)
    tc_or_skip(rc)
    H.assert_attn_close(out, ref, tb.node_off)


@pytest.mark.parametrize("tck", TC_KERNELS)
@pytest.mark.parametrize("T,G,L,splits", [(60, 1, 1024, 0), (60, 1, 700, 4), (80, 1, 500, 3), (16, 8, 1000, 5),
                                           (20, 1, 10, 2), (33, 2, 0, 1)])
def test_attn_tc_stable_prefix_flag_changes_nothing(T, G, L, splits, tck):
    """FALCON_ATTN_PREFIX_STABLE (prefix tiles requested before the preceding kernel has drained) leaves the
    output bit-identical, with the host copies it acts on and without them."""
    rng = np.random.default_rng(7000 + 100 * T + 10 * G + splits)
    Hkv = 2
    tb, q, k, v = random_case(rng, [T, max(1, T // 2)], [L, L // 3], Hkv * G, Hkv, 128, slack=1)
    ref = oracle_attn(tb, Hkv * G, Hkv, 128, q, k, v)
    dt = H.DevTrees(tb)
    base, rc = H.run_attn(dt, Hkv * G, Hkv, 128, q, k, v, kernel=tck, n_splits=splits, check=False,
                          host_copies=True)
    tc_or_skip(rc)
    H.assert_attn_close(base, ref, tb.node_off)
    for hc in (True, False):
        out, _ = H.run_attn(dt, Hkv * G, Hkv, 128, q, k, v, kernel=tck, n_splits=splits,
                            host_copies=hc, flags=binding.ATTN_PREFIX_STABLE)
        np.testing.assert_array_equal(out, base)
    assert not dt.status.cpu().numpy().any()


@pytest.mark.parametrize("tck", TC_KERNELS)
def test_attn_tc_stable_prefix_back_to_back_launches_match_single_launches(tck):
    """Eight layers launched back to back on one stream with the stable-prefix flag (each launch asks for
    its prefix tiles while the one before it is still finishing) give, bit for bit, what each layer gives
    when launched alone without the flag."""
    import torch
    spec = synth.SPECS["v7b"]
    tb = synth.make_trees(spec)
    dt = H.DevTrees(tb)
    Hq, Hkv, D = spec.n_q_heads, spec.n_kv_heads, spec.head_dim
    layers = [synth.make_layer_qkv(spec, tb, l) for l in range(8)]
    alone = []
    for q, k, v in layers:
        out, rc = H.run_attn(dt, Hq, Hkv, D, q, k, v, kernel=tck, check=False)
        tc_or_skip(rc)
        alone.append(out)
    dev = [(H.dev_bf16(q), H.dev_bf16(k), H.dev_bf16(v)) for q, k, v in layers]
    outs = [torch.full_like(q, float("nan")) for q, _, _ in dev]
    tree = dt.desc(host_copies=True)
    args = [binding.attn_args(tree, Hq, Hkv, D, 1.0 / np.sqrt(D), q, o, k, v, tuple(int(x) for x in k.stride()[:3]),
                              k.shape[2], kernel=tck, flags=binding.ATTN_PREFIX_STABLE)
            for (q, k, v), o in zip(dev, outs)]
    torch.cuda.synchronize()
    for _ in range(3):
        for a in args:
            H.ctx().falcon_tree_attn(a)
    torch.cuda.synchronize()
    for o, ref in zip(outs, alone):
        np.testing.assert_array_equal(H.host_bits(o), ref)
    assert not dt.status.cpu().numpy().any()


@pytest.mark.parametrize("tck", TC_KERNELS)
@pytest.mark.parametrize("seed", range(6))
def test_attn_tc_random_batches_and_splits(seed, tck):
    """Random batches (ragged trees and prefixes around the tile edges), head groupings and forced
    splits through the tensor-core kernel: oracle parity, bit-identical reruns, clean status words."""
    rng = np.random.default_rng(9000 + seed)
    for _ in range(6):
        G = int(rng.choice([1, 2, 4, 8]))
        Hkv = int(rng.choice([1, 2, 3]))
        B = int(rng.choice([1, 2, 3]))
        sizes = [int(rng.integers(1, 129)) for _ in range(B)]
        prefs = [int(rng.choice([0, 1, 63, 64, 65, int(rng.integers(0, 400))])) for _ in range(B)]
        splits = int(rng.choice([0, 1, 2, 3, 4, 5, 8]))
        tb, q, k, v = random_case(rng, sizes, prefs, Hkv * G, Hkv, 128, slack=int(rng.integers(0, 4)))
        ref = oracle_attn(tb, Hkv * G, Hkv, 128, q, k, v)
        dt = H.DevTrees(tb)
        hc = bool(rng.integers(0, 2))
        out, rc = H.run_attn(dt, Hkv * G, Hkv, 128, q, k, v, kernel=tck, n_splits=splits, check=False,
                             host_copies=hc)
        tc_or_skip(rc)
        H.assert_attn_close(out, ref, tb.node_off)
        again, _ = H.run_attn(dt, Hkv * G, Hkv, 128, q, k, v, kernel=tck, n_splits=splits, host_copies=hc)
        np.testing.assert_array_equal(out, again)
        assert not dt.status.cpu().numpy().any()


# ----------------------------------------------------------------------- top-m
@pytest.mark.parametrize("N,V,stride,m", [(1, 1, 1, 1), (3, 7, 9, 7), (5, 1000, 1000, 20), (60, 32000, 32000, 20),
                                          (4, 32001, 32005, 32), (2, 4099, 4101, 1), (2, 262144, 262144, 20),
                                          (130, 5000, 5000, 5), (3, 8192, 8192, 20), (70, 65536, 65536, 32),
                                          (9, 40000, 40000, 31)])
def test_topm_bit_exact(N, V, stride, m):
    rng = np.random.default_rng(V + m)
    x = rng.standard_normal((N, stride)).astype(np.float32)
    x[:, ::7] = np.round(x[:, ::7])                            # exact ties, also across chunk borders
    x[:, V:] = 1e9                                             # padding beyond the vocabulary is never read
    rv, ri = oracle.topm(x, m, vocab=V)
    for _ in range(2):                                         # twice: the arrival counters must come back to zero
        gv, gi, _ = H.run_topm(x, m, vocab=V)
        np.testing.assert_array_equal(gi, ri)
        np.testing.assert_array_equal(gv, rv)


def test_topm_ties_nan_inf_and_argmax_agreement():
    rng = np.random.default_rng(77)
    x = rng.standard_normal((6, 9000)).astype(np.float32)
    x[0, :] = 2.5                                              # all equal: indices 0..m-1
    x[1, 100:140] = np.nan
    x[1, 5000] = np.inf
    x[2, :] = -np.inf
    x[2, 8999] = np.nan                                        # counts as -inf: still indices 0..m-1
    x[3, 17] = 0.0
    x[3, 4] = -0.0
    x[3, :] = np.where(x[3] > 0, -x[3], x[3])                  # zeros are the maxima: index 4 (the -0) before 17
    x[3, 4], x[3, 17] = -0.0, 0.0
    x[4, 4095], x[4, 4096] = 50.0, 50.0                        # a tie across the chunk border
    rv, ri = oracle.topm(x, 20)
    gv, gi, _ = H.run_topm(x, 20)
    np.testing.assert_array_equal(gi, ri)
    np.testing.assert_array_equal(gv, rv)
    assert gi[0].tolist() == list(range(20)) and gi[2].tolist() == list(range(20))
    assert gi[3, :2].tolist() == [4, 17] and gi[4, :2].tolist() == [4095, 4096] and gi[1, 0] == 5000
    np.testing.assert_array_equal(H.run_topm(x, 1)[1][:, 0], oracle.argmax(x))


def test_topm_rejects_bad_arguments_without_launching():
    x = np.zeros((2, 64), np.float32)
    ld = torch.from_numpy(x).cuda()
    val = torch.full((2, 40), 3.0, dtype=torch.float32, device="cuda")
    idx = torch.full((2, 40), -7, dtype=torch.int32, device="cuda")
    for m, vocab in ((0, 64), (11, 10), (33, 64), (1, 0)):     # m < 1, m > vocab, m > FALCON_TOPM_MAX, empty rows
        rc = H.ctx().falcon_topm(binding.topm_args(2, vocab, ld, 64, m, val, idx), check=False)
        assert rc == binding.ERR_INVALID_ARG
    rc = H.ctx().falcon_topm(binding.topm_args(2, 64, ld, 32, 4, val, idx), check=False)   # stride < vocab
    assert rc == binding.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert (idx.cpu().numpy() == -7).all() and (val.cpu().numpy() == 3.0).all()


# ------------------------------------------------------------------------ non-greedy acceptance (Section 3.1)
SAMPLE_TOL = 1e-4   # fp32 partial sums of up to 32000 weights against the oracle's double ones, relative to the total


def assert_valid_draws(lg, vocab, T, u, g):
    """The kernel's token must be a valid inverse-CDF draw within fp32 rounding: the oracle's normalised partial
    sums just before and at the token bracket u up to SAMPLE_TOL, and the token has weight."""
    g_ref, cdf = oracle.sample_tokens(lg, T, u, vocab=vocab, want_cdf=True)
    N = len(g)
    assert g.min() >= 0 and g.max() < vocab
    hi = cdf[np.arange(N), g]
    lo = np.where(g > 0, cdf[np.arange(N), np.maximum(g - 1, 0)], 0.0)
    assert np.all(hi - lo > 0), "a token without weight was drawn"
    uu = u.astype(np.float64)
    assert np.all(lo <= uu + SAMPLE_TOL) and np.all(uu < hi + SAMPLE_TOL), (np.max(lo - uu), np.max(uu - hi))
    return g_ref


@pytest.mark.parametrize("name", ["tiny", "v7b", "l13b", "ragged"])
@pytest.mark.parametrize("T", [0.7, 1.0, 2.5])
def test_sample_accept_on_the_workloads(name, T):
    wl = synth.make_workload(name, with_logits=True)
    tb = wl.trees
    rng = np.random.default_rng(int(T * 10) + len(name))
    u = rng.random(tb.total_nodes).astype(np.float32)
    dt = H.DevTrees(tb)
    for _ in range(2):                                         # twice: both counters must come back to zero
        g, path, n_path, nxt = H.run_accept(dt, wl.logits, temperature=T, uniforms=u)
        g_ref = assert_valid_draws(wl.logits, wl.logits.shape[1], T, u, g)
        assert np.mean(g == g_ref) > 0.98
        rp, rn, rt = oracle.tree_accept(tb.node_off, tb.parent, tb.token, g)   # the search, given the drawn tokens
        np.testing.assert_array_equal(path, rp)
        np.testing.assert_array_equal(n_path, rn)
        np.testing.assert_array_equal(nxt, rt)


@pytest.mark.parametrize("V,stride", [(8192, 8192), (32000, 32000), (1000, 1003), (4097, 4100), (70000, 70000)])
def test_sample_equal_logits_are_bit_exact(V, stride):
    # equal logits: every weight is 1 and every partial sum an integer, exact in fp32; with u a multiple of 2^-10
    # u * V is exact too, so the token is floor(u * V) on both sides, boundaries included
    rng = np.random.default_rng(V)
    tb = H.make_trees([9, 30, 25], [3, 0, 8], rng, vocab=V)
    N = tb.total_nodes
    u = (rng.integers(0, 1024, N) / 1024.0).astype(np.float32)
    u[:4] = [0.0, 0.5, 1023.0 / 1024.0, 0.25]
    lg = np.full((N, stride), 1.25, dtype=np.float32)
    lg[:, V:] = 99.0                                           # padding beyond the vocabulary is never read
    g, path, n_path, nxt = H.run_accept(H.DevTrees(tb), lg, vocab=V, temperature=1.3, uniforms=u)
    np.testing.assert_array_equal(g, oracle.sample_tokens(lg, 1.3, u, vocab=V))
    np.testing.assert_array_equal(g, np.floor(u.astype(np.float64) * V).astype(np.int32))


def test_sample_edge_sizes_and_the_last_representable_uniform():
    rng = np.random.default_rng(41)
    for sizes, V in (([1], 1), ([1], 5), ([2, 1, 3], 4096), ([5], 4097), ([3], 12289)):
        tb = H.make_trees(sizes, [0] * len(sizes), rng, vocab=V)
        N = tb.total_nodes
        lg = rng.standard_normal((N, V)).astype(np.float32)
        u = rng.random(N).astype(np.float32)
        u[0] = np.float32(1.0) - np.float32(2.0 ** -24)        # the largest float below 1: the end of the row
        if N > 1:
            u[1] = 0.0                                         # the first token that has weight
        g = H.run_accept(H.DevTrees(tb), lg, temperature=0.9, uniforms=u)[0]
        assert_valid_draws(lg, V, 0.9, u, g)


def test_sample_special_values_and_the_greedy_limit():
    rng = np.random.default_rng(31)
    tb = H.make_trees([12, 20], [4, 4], rng, vocab=9000)
    N, V = tb.total_nodes, 9000
    dt = H.DevTrees(tb)
    u = rng.random(N).astype(np.float32)
    one = np.full((N, V), -np.inf, dtype=np.float32)
    pos = rng.integers(0, V, N)
    one[np.arange(N), pos] = rng.standard_normal(N).astype(np.float32)
    one[3, :] = np.nan                                         # nothing to draw from: 0
    one[4, 8000] = np.inf                                      # a +inf logit takes everything
    one[4, 8500] = np.inf
    g = H.run_accept(dt, one, temperature=1.0, uniforms=u)[0]
    exp = pos.copy()
    exp[3] = 0
    exp[4] = min(8000, pos[4]) if one[4, pos[4]] == np.inf else 8000
    np.testing.assert_array_equal(g, exp)
    np.testing.assert_array_equal(g, oracle.sample_tokens(one, 1.0, u))
    lg = rng.standard_normal((N, V)).astype(np.float32)
    lg[np.arange(N), pos] += 4.0                               # a clear maximum per row
    lg[:, ::97] = np.nan                                       # NaN entries have no weight
    lg[np.arange(N), pos] = np.where(np.isnan(lg[np.arange(N), pos]), 6.0, lg[np.arange(N), pos])
    cold = H.run_accept(dt, lg, temperature=1e-3, uniforms=u)
    greedy = H.run_accept(dt, lg)
    for a, b in zip(cold, greedy):                             # temperature -> 0: the greedy call's results
        np.testing.assert_array_equal(a, b)
    g = H.run_accept(dt, lg, temperature=1.0, uniforms=u)[0]
    assert not np.any(np.isnan(lg[np.arange(N), g]))
    assert_valid_draws(lg, V, 1.0, u, g)


def test_sample_rejects_bad_arguments():
    rng = np.random.default_rng(5)
    tb = H.make_trees([6], [2], rng, vocab=50)
    dt = H.DevTrees(tb)
    lg = torch.zeros((6, 50), dtype=torch.float32, device="cuda")
    u = torch.zeros(6, dtype=torch.float32, device="cuda")
    g = torch.zeros(6, dtype=torch.int32, device="cuda")
    path = torch.zeros((1, 8), dtype=torch.int32, device="cuda")
    n = torch.zeros(1, dtype=torch.int32, device="cuda")
    nxt = torch.zeros(1, dtype=torch.int32, device="cuda")
    c = H.ctx()

    def call(**kw):
        return binding.accept_args(dt.desc(), 50, lg, 50, g, path, 8, n, nxt, **kw)
    assert c.falcon_tree_accept(call(temperature=1.0, uniforms=u), check=False) == binding.OK
    assert c.falcon_tree_accept(call(temperature=1.0), check=False) == binding.ERR_INVALID_ARG
    assert c.falcon_tree_accept(call(temperature=-1.0, uniforms=u), check=False) == binding.ERR_INVALID_ARG
    assert c.falcon_tree_accept(call(temperature=float("nan"), uniforms=u), check=False) == binding.ERR_INVALID_ARG
    assert binding.falcon_tree_accept_static(call(temperature=1.0, uniforms=u), check=False) == binding.ERR_UNSUPPORTED
    torch.cuda.synchronize()


# ------------------------------------------------------------------------ the first launch of a process
FIRST_LAUNCH_SCRIPT = r"""
import sys
import numpy as np
sys.path.insert(0, sys.argv[1]); sys.path.insert(0, sys.argv[1] + "/tests")
import gpu_harness as H
from test_gpu_parity import random_case, oracle_attn
T, L, Hq, Hkv, splits, kernel = [int(x) for x in sys.argv[2:8]]
rng = np.random.default_rng(T + L)
tb, q, k, v = random_case(rng, [T], [L], Hq, Hkv, 128)
ref = oracle_attn(tb, Hq, Hkv, 128, q, k, v)
dt = H.DevTrees(tb)
out, rc = H.run_attn(dt, Hq, Hkv, 128, q, k, v, kernel=kernel, n_splits=splits)   # the process's first launch
assert rc == 0 and not dt.status.cpu().numpy().any()
H.assert_attn_close(out, ref, tb.node_off)
"""


@pytest.mark.parametrize("T,L,Hq,Hkv,splits,kernel", [(16, 112, 1, 1, 1, binding.ATTN_TCK), (60, 1024, 2, 2, 4, binding.ATTN_TCK),
                                                      (80, 300, 2, 2, 2, binding.ATTN_TCK), (128, 300, 2, 2, 3, binding.ATTN_TC)])
def test_first_launch_of_a_process_is_right(T, L, Hq, Hkv, splits, kernel):
    # every other test runs after earlier launches have warmed caches and left their data on the chip; here the
    # call under test is the very first kernel of a fresh process (a case that once showed a write into a tile
    # that the last MMAs were still reading, and only then)
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-c", FIRST_LAUNCH_SCRIPT, root] + [str(x) for x in (T, L, Hq, Hkv, splits, kernel)],
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]


# ------------------------------------------------------------------------ on-chip memory left by earlier launches
@pytest.mark.parametrize("pattern", [0xFFFFFFFF, 0x7F7F7F7F])
def test_results_do_not_depend_on_what_shared_and_tensor_memory_held(pattern):
    """Before every call the shared memory and the tensor memory of all SMs are filled with NaNs (all ones) or
    with huge finite numbers: a kernel that reads a tile row, an accumulator column or a scratch word it has not
    written itself computes with those instead of with what an earlier launch left, and shows it here."""
    rng = np.random.default_rng(2718)
    c = H.ctx()
    cases = [(binding.ATTN_TCK, [16], [112], 1, 1, 1), (binding.ATTN_TCK, [60], [68], 2, 2, 1),
             (binding.ATTN_TCK, [60], [300], 2, 2, 2), (binding.ATTN_TCK, [80], [700], 2, 2, 3),
             (binding.ATTN_TCK, [64], [900], 8, 1, 4), (binding.ATTN_TCK, [7, 33], [0, 130], 2, 2, 0),
             (binding.ATTN_TC, [60], [300], 2, 2, 2), (binding.ATTN_TC, [100], [40], 2, 1, 0),
             (binding.ATTN_WARP, [15], [128], 4, 4, 0), (binding.ATTN_SIMT, [20], [77], 2, 2, 0)]
    for kernel, sizes, prefs, Hq, Hkv, splits in cases:
        tb, q, k, v = random_case(rng, sizes, prefs, Hq, Hkv, 128)
        ref = oracle_attn(tb, Hq, Hkv, 128, q, k, v)
        dt = H.DevTrees(tb)
        c.falcon_test_poison(pattern)
        out, rc = H.run_attn(dt, Hq, Hkv, 128, q, k, v, kernel=kernel, n_splits=splits)
        assert rc == 0 and not dt.status.cpu().numpy().any()
        H.assert_attn_close(out, ref, tb.node_off)
    # the scan kernels and the LM head
    x = rng.standard_normal((9, 5000)).astype(np.float32)
    c.falcon_test_poison(pattern)
    gv, gi, _ = H.run_topm(x, 20)
    rv, ri = oracle.topm(x, 20)
    np.testing.assert_array_equal(gi, ri)
    np.testing.assert_array_equal(gv, rv)
    fi = rng.integers(-3, 4, size=(70, 192))
    wi = rng.integers(-3, 4, size=(1500, 192))
    f, w = synth.f32_to_bf16_bits(fi.astype(np.float32)), synth.f32_to_bf16_bits(wi.astype(np.float32))
    c.falcon_test_poison(pattern)
    g, mx, status, rc = H.run_lm_argmax(f, w)
    g_ref, best_ref = oracle.lm_head_argmax(f, w)
    assert rc == 0 and status == 0
    np.testing.assert_array_equal(g, g_ref)
    np.testing.assert_array_equal(mx.astype(np.float64), best_ref)
    tbt = H.make_trees([12, 30], [3, 9], rng, vocab=5000)
    lg = rng.standard_normal((tbt.total_nodes, 5000)).astype(np.float32)
    c.falcon_test_poison(pattern)
    g, path, n_path, nxt = H.run_accept(H.DevTrees(tbt), lg)
    np.testing.assert_array_equal(g, oracle.argmax(lg))
    rp, rn, rt = oracle.tree_accept(tbt.node_off, tbt.parent, tbt.token, g)
    np.testing.assert_array_equal(path, rp)
    np.testing.assert_array_equal(n_path, rn)


# ------------------------------------------------------------------------ LM-head argmax (Section 3.1, Eq. 6)
def assert_lm_argmax(f, w, hidden=None, tol=None):
    """The kernel sums in fp32 in the tensor core's order, the oracle in double: the maximum itself must agree
    within the rounding of those sums, and where the two pick different tokens the oracle's logit of the
    kernel's token must lie within that rounding of the oracle's maximum (both are then valid greedy tokens)."""
    g_ref, best_ref, logits = oracle.lm_head_argmax(f, w, hidden=hidden, want_logits=True)
    g, mx, status, rc = H.run_lm_argmax(f, w, hidden=hidden)
    assert rc == 0 and status == 0
    Hd = min(f.shape[1], w.shape[1]) if hidden is None else hidden
    if tol is None:
        # |sum error| <= hidden * 2^-24 * sum |a b| (fp32 accumulation of exact products), with slack 4
        fa = np.abs(synth.bf16_bits_to_f32(f[:, :Hd]).astype(np.float64))
        wa = np.abs(synth.bf16_bits_to_f32(w[:, :Hd]).astype(np.float64))
        tol = 4.0 * Hd * 2.0 ** -24 * float((fa.max(axis=0) * wa.max(axis=0)).sum())
    assert g.min() >= 0 and g.max() < w.shape[0]
    at_gpu = logits[np.arange(len(g)), g]
    assert np.all(best_ref - at_gpu <= tol), (np.max(best_ref - at_gpu), tol)
    assert np.all(np.abs(mx.astype(np.float64) - at_gpu) <= tol)
    return g, g_ref


@pytest.mark.parametrize("N,Hd,V", [(60, 256, 1000), (7, 64, 40), (130, 192, 3001), (300, 128, 2500), (60, 128, 50000),
                                    (1, 8, 1), (129, 64, 17), (2, 72, 2368), (64, 136, 2369)])
def test_lm_head_argmax_integer_data_is_bit_exact(N, Hd, V):
    # small integers: every product and every partial sum is exact in fp32, so values, ties and indices must
    # equal the oracle's bit for bit (one node tile, two resident tiles, three tiles in two rounds; a vocabulary
    # run longer than one MMA tile per CTA; vocabulary and node tails)
    rng = np.random.default_rng(N + V)
    fi = rng.integers(-3, 4, size=(N, Hd))
    wi = rng.integers(-3, 4, size=(V, Hd))
    if V > 8:
        wi[V // 2] = wi[5]                                     # identical head rows: a tie for every node
        wi[V - 1] = wi[5]
    f = synth.f32_to_bf16_bits(fi.astype(np.float32))
    w = synth.f32_to_bf16_bits(wi.astype(np.float32))
    g_ref, best_ref = oracle.lm_head_argmax(f, w)
    for _ in range(2):                                         # twice: the scratch must come back to zero
        g, mx, status, rc = H.run_lm_argmax(f, w)
        assert rc == 0 and status == 0
        np.testing.assert_array_equal(g, g_ref)
        np.testing.assert_array_equal(mx.astype(np.float64), best_ref)


@pytest.mark.parametrize("N,Hd,V,pad", [(60, 512, 5000, 0), (130, 320, 3001, 8), (15, 72, 1000, 24), (257, 256, 4096, 0)])
def test_lm_head_argmax_random_data(N, Hd, V, pad):
    # hidden sizes that are not multiples of the 64-column stage, padded row pitches, ragged tails
    rng = np.random.default_rng(N * 7 + V)
    f = synth.normal_bf16(rng, (N, Hd + pad))
    w = synth.normal_bf16(rng, (V, Hd + pad))
    g, g_ref = assert_lm_argmax(f, w, hidden=Hd)
    assert np.mean(g == g_ref) > 0.95                          # near-ties are rare with continuous data


def test_lm_head_argmax_full_size_7b_shape():
    # the size bench.py times: 60 nodes, hidden 4096, vocabulary 32000 (143 CTAs, 64 chunks of 64 columns each)
    rng = np.random.default_rng(2024)
    f = synth.normal_bf16(rng, (60, 4096))
    w = synth.normal_bf16(rng, (32000, 4096), std=0.02)
    g, g_ref = assert_lm_argmax(f, w)
    assert np.mean(g == g_ref) > 0.95


def test_lm_head_argmax_special_values():
    rng = np.random.default_rng(11)
    N, Hd, V = 20, 128, 700
    f = synth.normal_bf16(rng, (N, Hd))
    w = synth.normal_bf16(rng, (V, Hd))
    g0, _ = oracle.lm_head_argmax(f, w)
    wn = w.copy()
    wn[int(g0[0]), 3] = 0x7FC0                                 # the winner's head row gets a NaN: it cannot win
    g_ref, best_ref = oracle.lm_head_argmax(f, wn)
    g, mx, status, rc = H.run_lm_argmax(f, wn)
    assert rc == 0 and status == 0 and g[0] != g0[0]
    np.testing.assert_array_equal(g, g_ref)
    wn[:, 3] = 0x7FC0                                          # every logit NaN: index 0
    g, mx, status, rc = H.run_lm_argmax(f, wn)
    assert np.all(g == 0)
    z = np.zeros((4, Hd), dtype=np.uint16)                     # zero features: every logit is a zero, index 0
    z[1] = 0x8000
    g, mx, status, rc = H.run_lm_argmax(z, w)
    assert np.all(g == 0) and np.all(mx == 0.0)


def test_lm_head_argmax_then_accept_from_the_argmax():
    # verification without a logits matrix: the LM-head call writes g, the acceptance call with logits == NULL
    # searches the tree with it
    rng = np.random.default_rng(21)
    tb = H.make_trees([20, 33, 7], [5, 9, 0], rng, vocab=50)
    N, Hd, V = tb.total_nodes, 128, 50
    fi = rng.integers(-3, 4, size=(N, Hd))
    wi = rng.integers(-3, 4, size=(V, Hd))
    f = synth.f32_to_bf16_bits(fi.astype(np.float32))
    w = synth.f32_to_bf16_bits(wi.astype(np.float32))
    g_ref, _ = oracle.lm_head_argmax(f, w)
    for b in range(tb.batch):                                  # plant matches: a child carries its parent's argmax
        o = int(tb.node_off[b])
        for i in range(1, int(tb.node_off[b + 1]) - o):
            if rng.random() < 0.6:
                tb.token[o + i] = g_ref[o + tb.parent[o + i]]
    dt = H.DevTrees(tb)
    fd, wd = H.dev_bf16(f), H.dev_bf16(w)
    g = torch.zeros(N, dtype=torch.int32, device="cuda")
    path = torch.full((tb.batch, 64), -9, dtype=torch.int32, device="cuda")
    n_path = torch.zeros(tb.batch, dtype=torch.int32, device="cuda")
    nxt = torch.zeros(tb.batch, dtype=torch.int32, device="cuda")
    c = H.ctx()
    c.falcon_lm_head_argmax(binding.lm_argmax_args(N, Hd, V, fd, Hd, wd, Hd, g))
    c.falcon_tree_accept(binding.accept_args(dt.desc(), 0, None, 0, g, path, 64, n_path, nxt))
    torch.cuda.synchronize()
    np.testing.assert_array_equal(g.cpu().numpy(), g_ref)
    rp, rn, rt = oracle.tree_accept(tb.node_off, tb.parent, tb.token, g_ref, path_stride=64)
    np.testing.assert_array_equal(path.cpu().numpy(), rp)
    np.testing.assert_array_equal(n_path.cpu().numpy(), rn)
    np.testing.assert_array_equal(nxt.cpu().numpy(), rt)


def test_lm_head_argmax_bounded_wait_runs_out_and_the_context_stays_usable():
    # the test hook withholds the first stage's features: the MMA warp's wait gives up after its limit, every role
    # leaves in order, the status word says so, and the next call on the same context is right
    rng = np.random.default_rng(12)
    N, Hd, V = 40, 256, 3000
    fi = rng.integers(-3, 4, size=(N, Hd))
    wi = rng.integers(-3, 4, size=(V, Hd))
    f = synth.f32_to_bf16_bits(fi.astype(np.float32))
    w = synth.f32_to_bf16_bits(wi.astype(np.float32))
    fd, wd = H.dev_bf16(f), H.dev_bf16(w)
    g = torch.zeros(N, dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    c = H.ctx()
    rc = c.falcon_lm_head_argmax(binding.lm_argmax_args(N, Hd, V, fd, Hd, wd, Hd, g, None, st,
                                                        flags=binding.LM_TEST_STALL), check=False)
    torch.cuda.synchronize()
    assert rc == 0 and int(st.item()) & binding.DEV_TIMEOUT
    st.zero_()
    c.falcon_lm_head_argmax(binding.lm_argmax_args(N, Hd, V, fd, Hd, wd, Hd, g, None, st))
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    np.testing.assert_array_equal(g.cpu().numpy(), oracle.lm_head_argmax(f, w)[0])


def test_lm_head_argmax_rejects_bad_arguments_without_launching():
    f = torch.zeros((4, 72), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((10, 72), dtype=torch.bfloat16, device="cuda")
    g = torch.full((4,), -5, dtype=torch.int32, device="cuda")
    c = H.ctx()
    assert c.falcon_lm_head_argmax(binding.lm_argmax_args(4, 72, 10, f, 64, w, 72, g), check=False) == binding.ERR_INVALID_ARG
    assert c.falcon_lm_head_argmax(binding.lm_argmax_args(4, 70, 10, f, 70, w, 72, g), check=False) == binding.ERR_UNSUPPORTED
    assert c.falcon_lm_head_argmax(binding.lm_argmax_args(0, 72, 10, f, 72, w, 72, g), check=False) == binding.ERR_INVALID_ARG
    assert c.falcon_lm_head_argmax(binding.lm_argmax_args(4, 72, 10, f, 72, w, 72, None), check=False) == binding.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert (g.cpu().numpy() == -5).all()


# ------------------------------------------------------------------------ ABI
def test_abi_rejects_bad_arguments_without_launching():
    rng = np.random.default_rng(1)
    tb, q, k, v = random_case(rng, [8], [16], 2, 2, 128)
    dt = H.DevTrees(tb)
    qd, kd, vd = H.dev_bf16(q), H.dev_bf16(k), H.dev_bf16(v)
    out = torch.zeros_like(qd)
    st = tuple(int(s) for s in kd.stride()[:3])
    c = H.ctx()

    def attn(**kw):
        base = dict(tree=dt.desc(), n_q_heads=2, n_kv_heads=2, head_dim=128, sm_scale=0.1, q=qd, out=out, k_cache=kd,
                    v_cache=vd, strides=st, s_cap=24)
        base.update(kw)
        return c.falcon_tree_attn(binding.attn_args(**base), check=False)

    assert attn() == binding.OK
    assert attn(q=None) == binding.ERR_INVALID_ARG
    assert attn(head_dim=96) == binding.ERR_UNSUPPORTED
    assert attn(n_q_heads=3) == binding.ERR_UNSUPPORTED
    assert attn(strides=(st[0], st[1], 100)) == binding.ERR_INVALID_ARG
    assert attn(q=qd.data_ptr() + 2) == binding.ERR_INVALID_ARG
    assert attn(kernel=9) == binding.ERR_INVALID_ARG
    assert attn(n_splits=65) == binding.ERR_INVALID_ARG
    assert attn(k_tree=kd) == binding.ERR_INVALID_ARG          # k_tree without v_tree
    big = dt.desc()
    big.max_tree = 129
    assert attn(tree=big) == binding.ERR_UNSUPPORTED
    none = dt.desc()
    none.parent = None
    assert attn(tree=none) == binding.ERR_INVALID_ARG
    with pytest.raises(binding.FalconError):
        c.falcon_tree_attn(binding.attn_args(dt.desc(), 2, 2, 96, 0.1, qd, out, kd, vd, st, 24))

    lg = torch.zeros(8, 10, device="cuda")
    i32 = lambda *s: torch.zeros(*s, dtype=torch.int32, device="cuda")
    g, path, n, nxt = i32(8), i32(1, 128), i32(1), i32(1)
    assert c.falcon_tree_accept(binding.accept_args(dt.desc(), 10, lg, 10, g, path, 128, n, nxt), check=False) == 0
    assert c.falcon_tree_accept(binding.accept_args(dt.desc(), 10, lg, 9, g, path, 128, n, nxt), check=False) \
        == binding.ERR_INVALID_ARG
    assert c.falcon_tree_accept(binding.accept_args(dt.desc(), 0, lg, 10, g, path, 128, n, nxt), check=False) \
        == binding.ERR_INVALID_ARG
    assert c.falcon_tree_accept(binding.accept_args(dt.desc(), 10, lg, 10, g, path, 4, n, nxt), check=False) \
        == binding.ERR_INVALID_ARG
    assert c.falcon_tree_accept(binding.accept_args(dt.desc(), 10, lg, 10, None, path, 128, n, nxt), check=False) \
        == binding.ERR_INVALID_ARG                             # (logits == NULL alone is legal: g is then an input)
    torch.cuda.synchronize()


# ------------------------------------------------------------ contexts, scratch
def _accept_buffers(tb):
    i32 = lambda *s: torch.full(s, -7, dtype=torch.int32, device="cuda")
    return i32(tb.total_nodes), i32(tb.batch, 128), i32(tb.batch), i32(tb.batch)


def test_two_contexts_used_in_turn_keep_their_own_state():
    """Two contexts on the device, called alternately (attention through both tensor-core kernels, acceptance):
    launch attributes, cluster occupancy and scratch are per context, so neither disturbs the other."""
    import paper_2412_12639_b200 as falcon
    rng = np.random.default_rng(77)
    tb, q, k, v = random_case(rng, [60, 33], [700, 130], 4, 4, 128)
    ref = oracle_attn(tb, 4, 4, 128, q, k, v)
    logits = rng.standard_normal((tb.total_nodes, 5000)).astype(np.float32)
    g_ref = oracle.argmax(logits)
    p_ref, n_ref, t_ref = oracle.tree_accept(tb.node_off, tb.parent, tb.token, g_ref)
    dt = H.DevTrees(tb)
    qd, kd, vd, ld = H.dev_bf16(q), H.dev_bf16(k), H.dev_bf16(v), torch.from_numpy(logits).cuda()
    ctxs = [falcon.Context(0), falcon.Context(0)]
    strides = tuple(int(s) for s in kd.stride()[:3])
    for rnd in range(3):
        for c in ctxs:
            for kernel in TC_KERNELS:
                out = torch.full_like(qd, float("nan"))
                c.falcon_tree_attn(binding.attn_args(dt.desc(), 4, 4, 128, 1 / math.sqrt(128), qd, out, kd, vd, strides,
                                                     kd.shape[2], kernel=kernel))
                torch.cuda.synchronize()
                H.assert_attn_close(H.host_bits(out), ref, tb.node_off)
            g, path, n_path, nxt = _accept_buffers(tb)
            c.falcon_tree_accept(binding.accept_args(dt.desc(), 5000, ld, 5000, g, path, 128, n_path, nxt))
            torch.cuda.synchronize()
            np.testing.assert_array_equal(g.cpu().numpy(), g_ref)
            np.testing.assert_array_equal(path.cpu().numpy(), p_ref)
    for c in ctxs:
        c.close()


def test_captured_graph_survives_a_later_call_that_needs_more_scratch():
    """An acceptance call captured into a CUDA graph, then a top-m call on the same context that needs a larger
    scratch block and more arrival counters (on a non-blocking stream), then the graph replayed: the graph still
    names the block it was captured with, which must be alive and consistent."""
    import paper_2412_12639_b200 as falcon
    rng = np.random.default_rng(78)
    tb = H.make_trees([20, 9], [0, 0], rng, vocab=50)
    logits = rng.standard_normal((tb.total_nodes, 3000)).astype(np.float32)
    g_ref = oracle.argmax(logits)
    p_ref, n_ref, t_ref = oracle.tree_accept(tb.node_off, tb.parent, tb.token, g_ref)
    dt = H.DevTrees(tb)
    ld = torch.from_numpy(logits).cuda()
    c = falcon.Context(0)
    g, path, n_path, nxt = _accept_buffers(tb)
    acc = binding.accept_args(dt.desc(), 3000, ld, 3000, g, path, 128, n_path, nxt)
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        c.falcon_tree_accept(acc, stream=st)               # first call: allocates, outside the capture
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=st):
            c.falcon_tree_accept(acc, stream=st)
        big = torch.from_numpy(rng.standard_normal((300, 40000)).astype(np.float32)).cuda()
        val = torch.zeros((300, 8), device="cuda")
        idx = torch.zeros((300, 8), dtype=torch.int32, device="cuda")
        c.falcon_topm(binding.topm_args(300, 40000, big, 40000, 8, val, idx), stream=st)   # grows both scratch blocks
        for _ in range(3):
            g.fill_(-7)
            path.fill_(-7)
            graph.replay()
    torch.cuda.synchronize()
    np.testing.assert_array_equal(g.cpu().numpy(), g_ref)
    np.testing.assert_array_equal(path.cpu().numpy(), p_ref)
    np.testing.assert_array_equal(n_path.cpu().numpy(), n_ref)
    want_v, want_i = oracle.topm(big.cpu().numpy(), 8)
    np.testing.assert_array_equal(idx.cpu().numpy(), want_i)
    c.close()


@pytest.mark.parametrize("tck", TC_KERNELS)
@pytest.mark.parametrize("T", [60, 80])
def test_attn_bounded_wait_runs_out_and_the_context_stays_usable(tck, T):
    """The test hook FALCON_ATTN_TEST_STALL never requests a block's first key tile, so the wait for it runs out:
    the launch must return (no hang), report FALCON_DEV_TIMEOUT in the status word, leave finite rows (the
    keys-on-lanes kernel still delivers the right ones through its exact fallback path, the other kernel zeros),
    and the next ordinary launch on the same context must match the oracle."""
    rng = np.random.default_rng(4242 + T)
    tb, q, k, v = random_case(rng, [T], [400], 2, 2, 128)
    ref = oracle_attn(tb, 2, 2, 128, q, k, v)
    dt = H.DevTrees(tb)
    out, rc = H.run_attn(dt, 2, 2, 128, q, k, v, kernel=tck, n_splits=1, flags=binding.ATTN_TEST_STALL, check=False)
    tc_or_skip(rc)
    assert dt.status.cpu().numpy()[0] & binding.DEV_TIMEOUT
    got = synth.bf16_bits_to_f32(out)
    assert np.isfinite(got).all()
    if tck == binding.ATTN_TCK:
        H.assert_attn_close(out, ref, tb.node_off)
    else:
        assert not got.any()
    dt.status.zero_()
    out, _ = H.run_attn(dt, 2, 2, 128, q, k, v, kernel=tck)
    H.assert_attn_close(out, ref, tb.node_off)
    assert not dt.status.cpu().numpy().any()
    # the hook is refused where it would leave a cluster peer waiting, and on the other kernels
    for kw in ({"n_splits": 2, "kernel": tck}, {"n_splits": 1, "kernel": binding.ATTN_SIMT}, {"n_splits": 1}):
        _, rc = H.run_attn(dt, 2, 2, 128, q, k, v, flags=binding.ATTN_TEST_STALL, check=False, **kw)
        assert rc == binding.ERR_INVALID_ARG


# ------------------------------------------------- accepted tokens and features
def _gather_case(rng, sizes, hidden, stride_pad=0):
    tb = H.make_trees(sizes, [0] * len(sizes), rng, vocab=32000)
    N, B = tb.total_nodes, tb.batch
    feat = rng.integers(0, 65536, size=(N, hidden + stride_pad), dtype=np.uint16)
    path = np.full((B, 128), -1, np.int32)
    n_path = np.zeros(B, np.int32)
    for b, T in enumerate(sizes):                           # a real root-to-node chain of each tree
        node = int(rng.integers(0, T))
        chain = oracle.ancestors(tb.parent[tb.node_off[b]:tb.node_off[b + 1]], node)
        chain = sorted(chain)
        path[b, :len(chain)] = chain
        n_path[b] = len(chain)
    return tb, feat, path, n_path


@pytest.mark.parametrize("sizes,hidden,pad", [([6], 8, 0), ([60], 4096, 0), ([80, 1, 33], 5120, 8),
                                              ([128] * 3, 1024, 0), ([20, 80, 47, 64, 33, 21, 77, 50], 4096, 0)])
def test_feature_gather_bit_exact(sizes, hidden, pad):
    rng = np.random.default_rng(hidden + len(sizes))
    tb, feat, path, n_path = _gather_case(rng, sizes, hidden, pad)
    f_ref, t_ref = oracle.feature_gather(tb.node_off, path, n_path, tb.token, feat, hidden=hidden, fill=0x7777)
    dt = H.DevTrees(tb)
    fd = torch.from_numpy(feat.view(np.int16)).cuda()
    pd, nd = H.dev_i32(path), H.dev_i32(n_path)
    fo = torch.full((tb.batch, 128, hidden), 0x7777, dtype=torch.int16, device="cuda")
    to = torch.full((tb.batch, 128), 0x7777, dtype=torch.int32, device="cuda")
    a = binding.gather_args(dt.desc(), hidden, fd, feat.shape[1], pd, 128, nd, 128, fo, to)
    H.ctx().falcon_feature_gather(a)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(fo.cpu().numpy().view(np.uint16), f_ref)      # rows past the path untouched too
    np.testing.assert_array_equal(to.cpu().numpy(), t_ref)
    assert not dt.status.cpu().numpy().any()


def test_feature_gather_rides_on_the_compaction_launch():
    """falcon_kv_compact with `gather`: one launch compacts the caches and records the accepted tokens and features;
    both results equal the oracle's, bit for bit."""
    rng = np.random.default_rng(55)
    sizes, prefs, Hkv, D, hidden = [60, 17], [100, 31], 4, 128, 4096
    tb = H.make_trees(sizes, prefs, rng)
    s_cap = max(p + t for p, t in zip(prefs, sizes))
    k = [synth.normal_bf16(rng, (2, Hkv, s_cap, D)) for _ in range(3)]
    v = [synth.normal_bf16(rng, (2, Hkv, s_cap, D)) for _ in range(3)]
    logits = rng.standard_normal((tb.total_nodes, 50)).astype(np.float32)
    g = oracle.argmax(logits)
    path, n_path, _ = oracle.tree_accept(tb.node_off, tb.parent, tb.token, g)
    feat = rng.integers(0, 65536, size=(tb.total_nodes, hidden), dtype=np.uint16)
    f_ref, t_ref = oracle.feature_gather(tb.node_off, path, n_path, tb.token, feat, fill=0)
    dt = H.DevTrees(tb)
    kd, vd = [H.dev_bf16(x) for x in k], [H.dev_bf16(x) for x in v]
    kp = torch.tensor([t.data_ptr() for t in kd], dtype=torch.int64, device="cuda")
    vp = torch.tensor([t.data_ptr() for t in vd], dtype=torch.int64, device="cuda")
    pd, nd = H.dev_i32(path), H.dev_i32(n_path)
    new_len = torch.full((2,), -7, dtype=torch.int32, device="cuda")
    fd = torch.from_numpy(feat.view(np.int16)).cuda()
    fo = torch.zeros((2, 128, hidden), dtype=torch.int16, device="cuda")
    to = torch.zeros((2, 128), dtype=torch.int32, device="cuda")
    ga = binding.gather_args(dt.desc(), hidden, fd, hidden, pd, 128, nd, 128, fo, to)
    strides = tuple(int(s) for s in kd[0].stride()[:3])
    ca = binding.compact_args(dt.desc(), 3, Hkv, D, kp, vp, strides, s_cap, pd, 128, nd, new_len, gather=ga)
    H.ctx().falcon_kv_compact(ca)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(fo.cpu().numpy().view(np.uint16), f_ref)
    np.testing.assert_array_equal(to.cpu().numpy(), t_ref)
    st = strides_of(k[0])
    for layer in range(3):
        for host, devt in ((k[layer], kd[layer]), (v[layer], vd[layer])):
            ref = host.copy()
            nl = oracle.kv_compact(tb.node_off, tb.prefix_len, Hkv, D, ref, st, s_cap, path, n_path)
            got = H.host_bits(devt)
            for b in range(2):
                np.testing.assert_array_equal(got[b, :, :nl[b]], ref[b, :, :nl[b]])
            np.testing.assert_array_equal(new_len.cpu().numpy(), nl)
    assert not dt.status.cpu().numpy().any()


def test_feature_gather_bad_path_sets_status_and_writes_nothing():
    rng = np.random.default_rng(56)
    tb, feat, path, n_path = _gather_case(rng, [10, 12], 64)
    path[0, 1] = 11                                         # outside sequence 0's tree of 10 nodes
    n_path[0] = max(2, n_path[0])
    dt = H.DevTrees(tb)
    fd = torch.from_numpy(feat.view(np.int16)).cuda()
    fo = torch.full((2, 128, 64), 0x1111, dtype=torch.int16, device="cuda")
    to = torch.full((2, 128), -5, dtype=torch.int32, device="cuda")
    a = binding.gather_args(dt.desc(), 64, fd, 64, H.dev_i32(path), 128, H.dev_i32(n_path), 128, fo, to)
    H.ctx().falcon_feature_gather(a)
    torch.cuda.synchronize()
    st = dt.status.cpu().numpy()
    assert st[0] & binding.DEV_BAD_PATH and st[1] == 0
    assert (to.cpu().numpy()[0] == -5).all() and (fo.cpu().numpy()[0] == 0x1111).all()
    f_ref, t_ref = oracle.feature_gather(tb.node_off[1:] - tb.node_off[1], path[1:], n_path[1:], tb.token[10:], feat[10:])
    np.testing.assert_array_equal(to.cpu().numpy()[1, :n_path[1]], t_ref[0, :n_path[1]])
    # bad arguments are refused on the host
    bad = binding.gather_args(dt.desc(), 60, fd, 64, H.dev_i32(path), 128, H.dev_i32(n_path), 128, fo, to)
    assert H.ctx().falcon_feature_gather(bad, check=False) == binding.ERR_INVALID_ARG
