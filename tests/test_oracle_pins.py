"""Pins for the CPU oracle: closed forms, hand-worked trees, special cases that
reduce to library routines, brute force and invariants.  None of these values
comes from the CUDA path."""
import json
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2412_12639_b200 import synth

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "handworked.json")))


def bf(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def single_seq_cache(prefix_rows, tree_rows, Hkv=1):
    """[1, Hkv, L+T, D] cache (same rows for each head) from float rows."""
    rows = np.concatenate([np.asarray(prefix_rows, np.float32).reshape(-1, np.shape(tree_rows)[-1]),
                           np.asarray(tree_rows, np.float32)], axis=0)
    c = np.broadcast_to(rows[None, None], (1, Hkv) + rows.shape).copy()
    return bf(c)


def strides_of(cache):
    return tuple(s // 2 for s in cache.strides[:3])


def is_ancestor_or_self(parent, a, i):
    """Brute force, independent of the oracle: climb from i and look for a."""
    u = i
    while u != -1:
        if u == a:
            return True
        u = int(parent[u])
    return False


def dense_mask(parent, L):
    T = len(parent)
    m = np.zeros((T, L + T), dtype=bool)
    m[:, :L] = True
    for i in range(T):
        for a in range(T):
            m[i, L + a] = is_ancestor_or_self(parent, a, i)
    return m


# ----------------------------------------------------------------- attention
def test_attn_mean_of_visible_handworked():
    g = GOLD["attn_mean_of_visible"]
    parent = np.array(g["parent"], np.int32)
    T, L, D = len(parent), g["L"], g["D"]
    v = single_seq_cache(np.array(g["prefix_v"]).reshape(L, D), np.array(g["tree_v"]).reshape(T, D))
    k = bf(np.random.default_rng(0).standard_normal(v.shape))
    q = bf(np.zeros((T, 1, D)))
    out = oracle.tree_attn([0, T], parent, [L], 1, 1, D, 1.0, q, k, v, strides_of(k))
    np.testing.assert_allclose(out[:, 0, 0], g["expected"], rtol=0, atol=1e-7)


def test_attn_two_key_closed_form():
    g = GOLD["attn_two_keys"]
    k = single_seq_cache([[g["k"][0]]], [[g["k"][1]]])
    v = single_seq_cache([[g["v"][0]]], [[g["v"][1]]])
    q = bf(np.full((1, 1, 1), g["q"]))
    out = oracle.tree_attn([0, 1], [-1], [1], 1, 1, 1, 1.0, q, k, v, strides_of(k))
    expect = (g["v"][0] + math.e * g["v"][1]) / (1 + math.e)
    assert abs(out[0, 0, 0] - expect) < 1e-6
    # the scale multiplies the score: with sm_scale = 2 the weights are 1 and e^2
    out2 = oracle.tree_attn([0, 1], [-1], [1], 1, 1, 1, 2.0, q, k, v, strides_of(k))
    expect2 = (g["v"][0] + math.e ** 2 * g["v"][1]) / (1 + math.e ** 2)
    assert abs(out2[0, 0, 0] - expect2) < 1e-6


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_attn_indicator_values_read_back_visible_set(seed):
    rng = np.random.default_rng(seed)
    T, L = 23, 9
    parent = synth.random_tree(rng, T, 6, 3)
    D = L + T
    v = bf(np.eye(D, dtype=np.float32)[None, None])            # V[j] = e_j
    k = synth.normal_bf16(rng, (1, 1, D, D))
    q = bf(np.zeros((T, 1, D)))
    out = oracle.tree_attn([0, T], parent, [L], 1, 1, D, 0.3, q, k, v, strides_of(k))[:, 0]
    mask = dense_mask(parent, L)
    expect = mask / mask.sum(1, keepdims=True)
    np.testing.assert_allclose(out, expect, atol=1e-7)
    # depth + 1 tree keys are visible: prefix + ancestor chain, nothing else
    for i in range(T):
        assert mask[i].sum() == L + len(oracle.ancestors(parent, i))


def test_ancestors_walk_matches_brute_force():
    rng = np.random.default_rng(5)
    for _ in range(20):
        T = int(rng.integers(1, 129))
        parent = synth.random_shape_tree(rng, T)
        assert oracle.tree_validate(parent) == 0
        for i in range(T):
            chain = oracle.ancestors(parent, i)
            assert chain[0] == i and chain[-1] == 0
            assert sorted(chain.tolist()) == [a for a in range(T) if is_ancestor_or_self(parent, a, i)]


def test_tree_validate_rejects_malformed():
    assert oracle.tree_validate([-1, 0, 1]) == 0
    assert oracle.tree_validate([0, 0, 1]) == 1       # no root marker
    assert oracle.tree_validate([-1, 1, 0]) == 1      # self loop
    assert oracle.tree_validate([-1, 2, 1]) == 1      # parent after child
    assert oracle.tree_validate([-1, -1, 0]) == 1     # two roots


def test_attn_uniform_when_keys_identical_and_constant_values():
    rng = np.random.default_rng(3)
    T, L, D = 7, 5, 16
    parent = synth.random_tree(rng, T, 3, 3)
    krow = rng.standard_normal(D).astype(np.float32)
    k = bf(np.broadcast_to(krow, (1, 1, L + T, D)).copy())
    v = synth.normal_bf16(rng, (1, 1, L + T, D))
    q = synth.normal_bf16(rng, (T, 1, D))
    out = oracle.tree_attn([0, T], parent, [L], 1, 1, D, 0.25, q, k, v, strides_of(k))[:, 0]
    vf = synth.bf16_bits_to_f32(v)[0, 0].astype(np.float64)
    mask = dense_mask(parent, L)
    expect = (mask[:, :, None] * vf[None]).sum(1) / mask.sum(1, keepdims=True)
    np.testing.assert_allclose(out, expect, atol=1e-6)
    # constant V: normalisation must give exactly that row whatever q and K are
    vrow = bf(rng.standard_normal(D))
    v2 = np.broadcast_to(vrow, (1, 1, L + T, D)).copy()
    k2 = synth.normal_bf16(rng, (1, 1, L + T, D))
    out2 = oracle.tree_attn([0, T], parent, [L], 1, 1, D, 0.25, q, k2, v2, strides_of(k2))[:, 0]
    np.testing.assert_allclose(out2, np.broadcast_to(synth.bf16_bits_to_f32(vrow), (T, D)), atol=1e-6)


def sdpa_reference(q, k, v, mask, scale, G):
    """torch CPU scaled_dot_product_attention in float64 with an explicit mask.
    q [T,Hq,D] bits, k/v [Hkv,S,D] bits, mask [T,S] bool."""
    qt = torch.from_numpy(synth.bf16_bits_to_f32(q)).double().permute(1, 0, 2)          # [Hq,T,D]
    kt = torch.from_numpy(synth.bf16_bits_to_f32(k)).double().repeat_interleave(G, 0)   # [Hq,S,D]
    vt = torch.from_numpy(synth.bf16_bits_to_f32(v)).double().repeat_interleave(G, 0)
    o = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, attn_mask=torch.from_numpy(mask), scale=scale)
    return o.permute(1, 0, 2).numpy()


@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (4, 2), (8, 1)])
def test_attn_chain_tree_is_causal_attention(Hq, Hkv):
    rng = np.random.default_rng(11)
    T, L, D = 9, 13, 32
    parent = synth.chain_tree(T)
    q = synth.normal_bf16(rng, (T, Hq, D))
    k = synth.normal_bf16(rng, (1, Hkv, L + T, D))
    v = synth.normal_bf16(rng, (1, Hkv, L + T, D))
    scale = 1 / math.sqrt(D)
    out = oracle.tree_attn([0, T], parent, [L], Hq, Hkv, D, scale, q, k, v, strides_of(k))
    causal = oracle.causal_attn(L, T, Hq, Hkv, D, scale, q, k[0], v[0])
    np.testing.assert_allclose(out, causal, atol=2e-6)
    mask = np.tril(np.ones((T, L + T), dtype=bool), k=L)
    lib = sdpa_reference(q, k[0], v[0], mask, scale, Hq // Hkv)
    np.testing.assert_allclose(out, lib, atol=2e-6)


@pytest.mark.parametrize("seed", [0, 1])
def test_attn_random_tree_vs_library_sdpa_with_explicit_mask(seed):
    rng = np.random.default_rng(100 + seed)
    T, L, D, Hq, Hkv = 31, 40, 64, 4, 2
    parent = synth.random_tree(rng, T, 6, 4)
    q = synth.normal_bf16(rng, (T, Hq, D))
    k = synth.normal_bf16(rng, (1, Hkv, L + T + 3, D))   # 3 unused rows past the tree
    v = synth.normal_bf16(rng, (1, Hkv, L + T + 3, D))
    scale = 1 / math.sqrt(D)
    out = oracle.tree_attn([0, T], parent, [L], Hq, Hkv, D, scale, q, k, v, strides_of(k))
    lib = sdpa_reference(q, k[0, :, :L + T], v[0, :, :L + T], dense_mask(parent, L), scale, Hq // Hkv)
    np.testing.assert_allclose(out, lib, atol=2e-6)


def test_attn_single_node_is_plain_decode_attention():
    rng = np.random.default_rng(4)
    L, D, H = 50, 32, 3
    q = synth.normal_bf16(rng, (1, H, D))
    k = synth.normal_bf16(rng, (1, H, L + 1, D))
    v = synth.normal_bf16(rng, (1, H, L + 1, D))
    out = oracle.tree_attn([0, 1], [-1], [L], H, H, D, 0.2, q, k, v, strides_of(k))
    lib = sdpa_reference(q, k[0], v[0], np.ones((1, L + 1), dtype=bool), 0.2, 1)
    np.testing.assert_allclose(out, lib, atol=2e-6)


def test_attn_star_tree_sees_prefix_root_and_self_only():
    T, L = 21, 4       # root fan-out 20 (Appendix A: m = 20 at the root)
    parent = synth.star_tree(T)
    D = L + T
    v = bf(np.eye(D, dtype=np.float32)[None, None])
    k = bf(np.zeros((1, 1, D, D)))
    q = bf(np.zeros((T, 1, D)))
    out = oracle.tree_attn([0, T], parent, [L], 1, 1, D, 1.0, q, k, v, strides_of(k))[:, 0]
    for i in range(T):
        vis = set(range(L)) | {L, L + i}
        assert set(np.nonzero(out[i])[0].tolist()) == vis
        np.testing.assert_allclose(out[i][sorted(vis)], 1.0 / len(vis), atol=1e-7)


def test_attn_relabelling_nodes_permutes_rows():
    rng = np.random.default_rng(8)
    T, L, D = 17, 6, 16
    parent = synth.random_tree(rng, T, 5, 3)
    # another valid topological order: reverse the order inside each depth level
    depth = np.zeros(T, int)
    for i in range(1, T):
        depth[i] = depth[parent[i]] + 1
    order = sorted(range(T), key=lambda i: (depth[i], -i))     # new position -> old node
    new_of_old = np.empty(T, int)
    new_of_old[order] = np.arange(T)
    parent2 = np.array([-1 if parent[o] < 0 else new_of_old[parent[o]] for o in order], np.int32)
    assert oracle.tree_validate(parent2) == 0
    q = synth.normal_bf16(rng, (T, 1, D))
    k = synth.normal_bf16(rng, (1, 1, L + T, D))
    v = synth.normal_bf16(rng, (1, 1, L + T, D))
    k2, v2 = k.copy(), v.copy()
    k2[0, 0, L:] = k[0, 0, L:][order]
    v2[0, 0, L:] = v[0, 0, L:][order]
    out = oracle.tree_attn([0, T], parent, [L], 1, 1, D, 0.25, q, k, v, strides_of(k))
    out2 = oracle.tree_attn([0, T], parent2, [L], 1, 1, D, 0.25, q[order], k2, v2, strides_of(k))
    np.testing.assert_allclose(out2, out[order], atol=1e-6)


def test_attn_gqa_head_mapping_and_batch_packing():
    rng = np.random.default_rng(9)
    Hq, Hkv, D = 6, 3, 8
    sizes, prefs = [3, 5], [2, 4]
    node_off = np.array([0, 3, 8], np.int32)
    parent = np.concatenate([synth.random_tree(rng, t, 3, 2) for t in sizes])
    s_cap = 10
    k = synth.normal_bf16(rng, (2, Hkv, s_cap, D))
    # V constant per (sequence, kv head): the output must equal that constant for heads h with h // G == kvh
    const = rng.integers(-8, 8, size=(2, Hkv)).astype(np.float32)
    v = bf(np.broadcast_to(const[:, :, None, None], (2, Hkv, s_cap, D)).copy())
    q = synth.normal_bf16(rng, (8, Hq, D))
    out = oracle.tree_attn(node_off, parent, prefs, Hq, Hkv, D, 0.5, q, k, v, strides_of(k))
    for b in range(2):
        for h in range(Hq):
            np.testing.assert_allclose(out[node_off[b]:node_off[b + 1], h], const[b, h // 2], atol=1e-6)


def test_attn_separate_tree_buffers_equal_in_cache_rows():
    rng = np.random.default_rng(10)
    Hq, Hkv, D = 4, 2, 16
    node_off = np.array([0, 6, 10], np.int32)
    prefs = np.array([5, 0], np.int32)                     # second sequence has an empty prefix
    parent = np.concatenate([synth.random_tree(rng, 6, 3, 3), synth.random_tree(rng, 4, 2, 2)])
    s_cap = 12
    k = synth.normal_bf16(rng, (2, Hkv, s_cap, D))
    v = synth.normal_bf16(rng, (2, Hkv, s_cap, D))
    q = synth.normal_bf16(rng, (10, Hq, D))
    ref = oracle.tree_attn(node_off, parent, prefs, Hq, Hkv, D, 0.25, q, k, v, strides_of(k))
    kt = np.empty((10, Hkv, D), np.uint16)
    vt = np.empty((10, Hkv, D), np.uint16)
    k_nt, v_nt = k.copy(), v.copy()
    for b in range(2):
        L, T = prefs[b], node_off[b + 1] - node_off[b]
        kt[node_off[b]:node_off[b + 1]] = k[b, :, L:L + T].transpose(1, 0, 2)
        vt[node_off[b]:node_off[b + 1]] = v[b, :, L:L + T].transpose(1, 0, 2)
        k_nt[b, :, L:] = 0x7FC0      # NaN where the tree rows used to be
        v_nt[b, :, L:] = 0x7FC0
    out = oracle.tree_attn(node_off, parent, prefs, Hq, Hkv, D, 0.25, q, k_nt, v_nt, strides_of(k), kt, vt)
    np.testing.assert_array_equal(out, ref)


def test_attn_explicit_mask_rows_reproduce_the_ancestor_mask():
    rng = np.random.default_rng(12)
    T, L, D = 70, 3, 8
    parent = synth.random_tree(rng, T, 8, 4)
    q = synth.normal_bf16(rng, (T, 1, D))
    k = synth.normal_bf16(rng, (1, 1, L + T, D))
    v = synth.normal_bf16(rng, (1, 1, L + T, D))
    rows = np.zeros((T, 2), np.uint64)
    for i in range(T):
        for a in range(T):
            if is_ancestor_or_self(parent, a, i):
                rows[i, a >> 6] |= np.uint64(1) << np.uint64(a & 63)
    a = oracle.tree_attn([0, T], parent, [L], 1, 1, D, 0.3, q, k, v, strides_of(k))
    b = oracle.tree_attn([0, T], parent, [L], 1, 1, D, 0.3, q, k, v, strides_of(k), tree_mask=rows)
    np.testing.assert_allclose(a, b, atol=1e-7)


def test_attn_mask_rows_on_a_batch_match_sdpa_with_the_same_boolean_mask():
    """The caller-supplied mask branch against torch's scaled_dot_product_attention with an explicit boolean mask,
    on two sequences of different tree size and prefix length: rows of the drafter's relaxed causal mask
    (Section 3.4: predecessors in the tree plus the node's own k-block) and one row with an ancestor bit cleared.
    A wrong row offset for the second sequence, or rows merged with the ancestor chain, fail here."""
    import torch
    rng = np.random.default_rng(33)
    sizes, prefs, Hq, Hkv, D, kblk = [23, 70], [5, 41], 4, 2, 16, 3
    node_off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    parents = [synth.random_tree(rng, t, 8, 4) for t in sizes]
    parent = np.concatenate(parents).astype(np.int32)
    N, s_cap = int(node_off[-1]), max(p + t for p, t in zip(prefs, sizes)) + 1
    q = synth.normal_bf16(rng, (N, Hq, D))
    k = synth.normal_bf16(rng, (2, Hkv, s_cap, D))
    v = synth.normal_bf16(rng, (2, Hkv, s_cap, D))
    rows = np.zeros((N, 2), np.uint64)
    vis = [[set() for _ in range(t)] for t in sizes]
    for b, (T, par) in enumerate(zip(sizes, parents)):
        for i in range(T):
            s_ = {a for a in range(T) if is_ancestor_or_self(par, a, i)} | set(range(i - i % kblk, min(T, i - i % kblk + kblk)))
            vis[b][i] = s_
    dropped = int(parents[1][40])
    vis[1][40].discard(dropped)                                # not even the ancestor chain is implied
    for b, T in enumerate(sizes):
        for i in range(T):
            for a in vis[b][i]:
                rows[node_off[b] + i, a >> 6] |= np.uint64(1) << np.uint64(a & 63)
    out = oracle.tree_attn(node_off, parent, prefs, Hq, Hkv, D, 0.31, q, k, v, strides_of(k), tree_mask=rows)
    plain = oracle.tree_attn(node_off, parent, prefs, Hq, Hkv, D, 0.31, q, k, v, strides_of(k))
    assert np.abs(out - plain).max() > 1e-2
    qf, kf, vf = (torch.from_numpy(synth.bf16_bits_to_f32(x).astype(np.float64)) for x in (q, k, v))
    G = Hq // Hkv
    for b, (T, L) in enumerate(zip(sizes, prefs)):
        mask = torch.zeros(T, L + T, dtype=torch.bool)
        mask[:, :L] = True
        for i in range(T):
            for a in vis[b][i]:
                mask[i, L + a] = True
        for h in range(Hq):
            qq = qf[node_off[b]:node_off[b + 1], h]
            want = torch.nn.functional.scaled_dot_product_attention(
                qq[None], kf[b, h // G, :L + T][None], vf[b, h // G, :L + T][None], attn_mask=mask[None], scale=0.31)[0]
            np.testing.assert_allclose(out[node_off[b]:node_off[b + 1], h], want.numpy(), atol=2e-6, rtol=1e-6)


# -------------------------------------------------------------------- argmax
def test_argmax_planted_ties_and_special_values():
    rng = np.random.default_rng(0)
    for V in (1, 7, 1000, 32000, 32001):
        x = rng.standard_normal((5, V)).astype(np.float32)
        want = rng.integers(0, V, size=5)
        for i, w in enumerate(want):
            x[i, w] = 50.0
        np.testing.assert_array_equal(oracle.argmax(x), want)
        np.testing.assert_array_equal(oracle.argmax(x), np.argmax(x, axis=1))
    x = np.zeros((4, 9), np.float32)
    x[0, [3, 6]] = 2.0                                   # tie: lower index
    x[1] = [-0.0, 0.0, -0.0, 0.0, 0, 0, 0, 0, 0]         # +0 == -0: index 0
    x[2] = np.nan                                        # all NaN: 0
    x[3] = -np.inf                                       # all -inf: 0
    np.testing.assert_array_equal(oracle.argmax(x), [3, 0, 0, 0])
    y = np.array([[np.nan, 1.0, np.nan, 5.0, np.nan, 5.0]], np.float32)
    np.testing.assert_array_equal(oracle.argmax(y), [3])  # NaN never wins
    # padded rows: only the first `vocab` columns count
    z = np.zeros((2, 8), np.float32)
    z[:, 7] = 9.0
    z[0, 2] = 1.0
    np.testing.assert_array_equal(oracle.argmax(z, vocab=6), [2, 0])


# ---------------------------------------------------------------- acceptance
@pytest.mark.parametrize("case", ["accept_basic", "accept_root_only", "accept_duplicate_siblings",
                                  "accept_tie_lowest_index"])
def test_accept_handworked(case):
    g = GOLD[case]
    T = len(g["parent"])
    for fn in (oracle.tree_accept, oracle.bruteforce_accept):
        path, n_path, nxt = fn([0, T], g["parent"], g["token"], g["g"], path_stride=8)
        assert n_path[0] == g["n_path"]
        assert path[0, :n_path[0]].tolist() == g["path"]
        assert (path[0, n_path[0]:] == -1).all()
        assert nxt[0] == g["next_token"]


def check_accept_invariants(parent, token, g, path, n):
    T = len(parent)
    assert path[0] == 0 and 1 <= n <= T
    depth = np.zeros(T, int)
    alive = np.zeros(T, bool)
    alive[0] = True
    for c in range(1, T):
        depth[c] = depth[parent[c]] + 1
        alive[c] = alive[parent[c]] and token[c] == g[parent[c]]
    for j in range(n - 1):
        assert parent[path[j + 1]] == path[j]                 # prefix-closed ancestor chain
        assert token[path[j + 1]] == g[path[j]]               # every step is an accepted draft
    last = path[n - 1]
    assert alive[last] and depth[last] == n - 1
    assert not (alive & (depth > depth[last])).any()          # nothing alive is deeper
    assert not (alive & (depth == depth[last]) & (np.arange(T) < last)).any()   # tie -> lowest index


@pytest.mark.parametrize("seed", range(6))
def test_accept_matches_bruteforce_and_invariants_on_random_trees(seed):
    rng = np.random.default_rng(seed)
    B = 12
    sizes = [int(rng.integers(1, 129)) for _ in range(B)]
    node_off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    vocab = 6                                                  # tiny vocab: many matches and duplicate siblings
    parent = np.concatenate([synth.random_shape_tree(rng, t) for t in sizes])
    token = rng.integers(0, vocab, size=node_off[-1]).astype(np.int32)
    g = rng.integers(0, vocab, size=node_off[-1]).astype(np.int32)
    p1, n1, t1 = oracle.tree_accept(node_off, parent, token, g)
    p2, n2, t2 = oracle.bruteforce_accept(node_off, parent, token, g)
    np.testing.assert_array_equal(p1, p2)
    np.testing.assert_array_equal(n1, n2)
    np.testing.assert_array_equal(t1, t2)
    for b in range(B):
        lo, hi = node_off[b], node_off[b + 1]
        check_accept_invariants(parent[lo:hi], token[lo:hi], g[lo:hi], p1[b], n1[b])
        assert t1[b] == g[lo + p1[b, n1[b] - 1]]


def test_accept_chain_stops_at_first_mismatch():
    T = 9
    parent = synth.chain_tree(T)
    g = np.arange(100, 100 + T).astype(np.int32)
    for first_bad in range(1, T + 1):
        token = np.zeros(T, np.int32)
        token[1:] = g[:-1]
        if first_bad < T:
            token[first_bad] = -5
        path, n, nxt = oracle.tree_accept([0, T], parent, token, g)
        assert n[0] == first_bad and path[0, :n[0]].tolist() == list(range(first_bad))
        assert nxt[0] == g[first_bad - 1]


def test_planted_logits_give_plausible_acceptance_lengths():
    # sanity only: planting with p = 0.7 on depth-6 trees gives a mean accepted length between 0.7 and the
    # geometric bound sum_{d=1..6} 0.7^d = 2.06
    spec = synth.SPECS["v7b"]
    lens = []
    for seed in range(12):
        tb = synth.make_trees(spec, seed)
        lg = synth.make_logits(spec, tb, seed)
        g = oracle.argmax(lg)
        _, n, _ = oracle.tree_accept(tb.node_off, tb.parent, tb.token, g)
        lens.append(n[0] - 1)
    assert 0.7 <= np.mean(lens) <= 2.2


# ---------------------------------------------------------------- compaction
def test_compact_handworked_overlap():
    g = GOLD["compact_overlap"]
    L, T, D = g["L"], g["T"], 4
    rows = np.array(g["rows_before"], np.uint16)
    cache = np.broadcast_to(rows[None, None, :, None], (1, 2, L + T, D)).copy()
    path = np.array([g["path"] + [-1]], np.int32)
    new_len = oracle.kv_compact([0, T], [L], 2, D, cache, strides_of(cache), L + T, path, [len(g["path"])])
    assert new_len[0] == g["new_len"]
    assert cache[0, 0, :new_len[0], 0].tolist() == g["rows_after_valid"]
    assert cache[0, 1, :new_len[0], 3].tolist() == g["rows_after_valid"]


@pytest.mark.parametrize("seed", range(4))
def test_compact_is_a_gather_of_accepted_rows(seed):
    rng = np.random.default_rng(seed)
    B, Hkv, D = 3, 2, 8
    sizes = [int(rng.integers(1, 40)) for _ in range(B)]
    prefs = np.array([int(rng.integers(0, 20)) for _ in range(B)], np.int32)
    node_off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    s_cap = int(prefs.max()) + max(sizes) + 2
    cache = rng.integers(0, 65536, size=(B, Hkv, s_cap, D)).astype(np.uint16)
    before = cache.copy()
    path = np.full((B, 128), -1, np.int32)
    n_path = np.zeros(B, np.int32)
    for b in range(B):
        parent = synth.random_tree(rng, sizes[b], 6, 3)
        chain = oracle.ancestors(parent, int(rng.integers(0, sizes[b])))[::-1]
        path[b, :len(chain)] = chain
        n_path[b] = len(chain)
    new_len = oracle.kv_compact(node_off, prefs, Hkv, D, cache, strides_of(cache), s_cap, path, n_path)
    tree_rows = np.empty((node_off[-1], Hkv, D), np.uint16)
    for b in range(B):
        L = prefs[b]
        assert new_len[b] == L + n_path[b]
        np.testing.assert_array_equal(cache[b, :, :L], before[b, :, :L])              # prefix untouched
        gathered = before[b][:, L + path[b, :n_path[b]]]
        np.testing.assert_array_equal(cache[b, :, L:new_len[b]], gathered)            # gather of accepted rows
        tree_rows[node_off[b]:node_off[b + 1]] = before[b, :, L:L + sizes[b]].transpose(1, 0, 2)
    # separate tree buffer variant gives the same valid rows
    cache2 = before.copy()
    for b in range(B):
        cache2[b, :, prefs[b]:] = 0xDEAD
    oracle.kv_compact(node_off, prefs, Hkv, D, cache2, strides_of(cache2), s_cap, path, n_path, tree_rows=tree_rows)
    for b in range(B):
        np.testing.assert_array_equal(cache2[b, :, :new_len[b]], cache[b, :, :new_len[b]])


def test_compact_identity_path_is_a_no_op():
    rng = np.random.default_rng(1)
    T, L = 6, 3
    cache = rng.integers(0, 65536, size=(1, 1, L + T, 4)).astype(np.uint16)
    before = cache.copy()
    path = np.arange(T, dtype=np.int32)[None]
    oracle.kv_compact([0, T], [L], 1, 4, cache, strides_of(cache), L + T, path, [T])
    np.testing.assert_array_equal(cache, before)


# ------------------------------------------------------------------ generator
def test_generator_trees_respect_limits():
    for name, spec in synth.SPECS.items():
        tb = synth.make_trees(spec)
        for b in range(tb.batch):
            par = tb.parent[tb.node_off[b]:tb.node_off[b + 1]]
            T = len(par)
            assert oracle.tree_validate(par) == 0
            depth = np.zeros(T, int)
            for i in range(1, T):
                depth[i] = depth[par[i]] + 1
            assert depth.max() <= spec.max_depth
            assert np.bincount(par[1:], minlength=T).max() <= spec.branch
            if spec.tree is not None:
                assert T == spec.tree and depth.max() == min(spec.max_depth, T - 1)
    a = synth.make_trees(synth.SPECS["ragged"])
    b = synth.make_trees(synth.SPECS["ragged"])
    np.testing.assert_array_equal(a.parent, b.parent)           # seeded: reproducible
    assert a.batch == 8 and 256 <= a.prefix_len.min() and a.prefix_len.max() <= 4096


def test_bf16_bit_conversion_round_trip_and_rounding():
    x = np.array([1.0, -2.5, 0.0, 3.140625, 1e-3], np.float32)
    bits = synth.f32_to_bf16_bits(x)
    t = torch.from_numpy(x).to(torch.bfloat16)
    np.testing.assert_array_equal(bits, t.view(torch.int16).numpy().view(np.uint16))
    np.testing.assert_array_equal(synth.bf16_bits_to_f32(bits), t.float().numpy())
    y = np.random.default_rng(0).standard_normal(10000).astype(np.float32)
    np.testing.assert_array_equal(synth.f32_to_bf16_bits(y),
                                  torch.from_numpy(y).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))


# ------------------------------------------------------------------ top-m selection (Appendix A)
def test_topm_matches_a_stable_library_sort():
    # second opinion: numpy's stable argsort of the negated row gives the same order (lower index first among equals)
    rng = np.random.default_rng(3)
    for V, m in ((1, 1), (7, 7), (1000, 20), (32001, 20), (4099, 32)):
        x = rng.standard_normal((4, V)).astype(np.float32)
        x[:, ::5] = np.round(x[:, ::5])                       # plenty of exact ties
        val, idx = oracle.topm(x, m)
        ref = np.argsort(-x, axis=1, kind="stable")[:, :m]
        np.testing.assert_array_equal(idx, ref)
        np.testing.assert_array_equal(val, np.take_along_axis(x, ref, 1))


def test_topm_with_torch_topk_values_and_first_entry_is_argmax():
    rng = np.random.default_rng(4)
    x = rng.standard_normal((6, 5000)).astype(np.float32)
    val, idx = oracle.topm(x, 20)
    tv, _ = torch.topk(torch.from_numpy(x), 20, dim=1)        # values are unique up to ties; indices may differ on ties
    np.testing.assert_array_equal(val, tv.numpy())
    np.testing.assert_array_equal(idx[:, 0], oracle.argmax(x))


def test_topm_hand_worked_ties_zero_signs_and_nan():
    # row: values              index: 0    1     2    3     4    5        6
    x = np.array([[1.0, 3.0, 3.0, -0.0, 0.0, np.nan, -np.inf]], np.float32)
    val, idx = oracle.topm(x, 7)
    # 3 (index 1 before 2), 1, then the zeros as equals (index 3 before 4), then -inf entries by index: the NaN at 5
    # counts as -inf and comes before the real -inf at 6
    assert idx[0].tolist() == [1, 2, 0, 3, 4, 5, 6]
    assert val[0, :3].tolist() == [3.0, 3.0, 1.0] and np.all(val[0, 3:5] == 0.0)
    assert np.isneginf(val[0, 5]) and np.isneginf(val[0, 6])
    # a descending row returns 0..m-1, an ascending one V-1..V-m
    d = np.arange(50, 0, -1, dtype=np.float32)[None]
    assert oracle.topm(d, 5)[1][0].tolist() == [0, 1, 2, 3, 4]
    assert oracle.topm(d[:, ::-1].copy(), 5)[1][0].tolist() == [49, 48, 47, 46, 45]
    with pytest.raises(ValueError):
        oracle.topm(d, 51)


def test_topm_respects_row_stride_and_permutations():
    rng = np.random.default_rng(5)
    V, stride, m = 777, 800, 12
    buf = rng.standard_normal((3, stride)).astype(np.float32)
    buf[:, V:] = 100.0                                         # padding must never be selected
    val, idx = oracle.topm(buf, m, vocab=V)
    assert idx.max() < V
    perm = rng.permutation(V)
    shuffled = buf.copy()
    shuffled[:, :V] = buf[:, :V][:, perm]
    val2, idx2 = oracle.topm(shuffled, m, vocab=V)
    np.testing.assert_array_equal(val, val2)                   # the values are a property of the multiset
    np.testing.assert_array_equal(perm[idx2], idx)             # distinct values almost surely: indices map back


# ------------------------------------------------------------ feature gather
def test_feature_gather_hand_worked():
    case = GOLD["feature_gather_basic"]
    T, Hd = len(case["parent"]), case["hidden"]
    feat = np.array([[10 * i + c for c in range(Hd)] for i in range(T)], np.uint16)
    path = np.full((1, 8), -1, np.int32)
    path[0, :3] = case["path"]
    fo, to = oracle.feature_gather([0, T], path, [case["n_path"]], case["token"], feat, fill=777)
    np.testing.assert_array_equal(to[0, :3], case["expected_tokens"])
    np.testing.assert_array_equal(fo[0, :3], np.array(case["expected_features"], np.uint16))
    assert (to[0, 3:] == 777).all() and (fo[0, 3:] == 777).all()        # rows past the path are not touched


def test_feature_gather_equals_fancy_indexing_on_random_batches():
    rng = np.random.default_rng(91)
    for _ in range(20):
        B = int(rng.integers(1, 5))
        sizes = [int(rng.integers(1, 129)) for _ in range(B)]
        node_off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
        N, Hd = int(node_off[-1]), int(rng.choice([8, 40, 128]))
        feat = rng.integers(0, 65536, size=(N, Hd + 8), dtype=np.uint16)       # row stride wider than hidden
        token = rng.integers(0, 32000, size=N).astype(np.int32)
        path = np.full((B, 128), -1, np.int32)
        n_path = np.zeros(B, np.int32)
        for b, T in enumerate(sizes):
            n = int(rng.integers(1, T + 1))
            path[b, :n] = np.sort(rng.choice(T, size=n, replace=False))     # any increasing node list will do here
            n_path[b] = n
        fo, to = oracle.feature_gather(node_off, path, n_path, token, feat, hidden=Hd, fill=9)
        for b in range(B):
            idx = node_off[b] + path[b, :n_path[b]]
            np.testing.assert_array_equal(fo[b, :n_path[b]], feat[idx, :Hd])
            np.testing.assert_array_equal(to[b, :n_path[b]], token[idx])
            assert (fo[b, n_path[b]:] == 9).all() and (to[b, n_path[b]:] == 9).all()


def test_feature_gather_rejects_bad_paths():
    feat = np.zeros((4, 8), np.uint16)
    path = np.array([[0, 7, -1, -1]], np.int32)                                # node 7 is outside a tree of 4
    with pytest.raises(ValueError):
        oracle.feature_gather([0, 4], path, [2], [1, 2, 3, 4], feat)
    with pytest.raises(ValueError):
        oracle.feature_gather([0, 4], np.array([[0, 1, 2, 3]], np.int32), [5], [1, 2, 3, 4], feat)


# --------------------------------------------------------------------------- LM-head argmax (Section 3.1, Eq. 6)
def _bits(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def test_lm_head_argmax_hand_worked():
    c = GOLD["lm_head_argmax_basic"]
    g, best, logits = oracle.lm_head_argmax(_bits(c["features"]), _bits(c["head"]), want_logits=True)
    assert np.array_equal(logits, np.array(c["expected_logits"], dtype=np.float64))
    assert g.tolist() == c["expected_argmax"]          # node 0: three-way tie, the lowest index wins
    assert best.tolist() == c["expected_best"]


def test_lm_head_logits_are_the_matrix_product_with_the_head_transposed():
    rng = np.random.default_rng(3)
    N, H, V = 7, 96, 53                                 # all different: a transposed operand cannot pass
    f = synth.normal_bf16(rng, (N, H))
    w = synth.normal_bf16(rng, (V, H))
    g, best, logits = oracle.lm_head_argmax(f, w, want_logits=True)
    ref = synth.bf16_bits_to_f32(f).astype(np.float64) @ synth.bf16_bits_to_f32(w).astype(np.float64).T
    assert np.allclose(logits, ref, rtol=1e-12, atol=1e-12)
    assert np.array_equal(g, np.argmax(ref, axis=1))
    assert np.array_equal(best, logits[np.arange(N), g])


def test_lm_head_integer_data_is_exact_and_ties_go_to_the_lowest_index():
    rng = np.random.default_rng(4)
    N, H, V = 9, 64, 40
    fi = rng.integers(-3, 4, size=(N, H))
    wi = rng.integers(-3, 4, size=(V, H))
    wi[17] = wi[5]                                      # two identical head rows: equal logits for every node
    g, best, logits = oracle.lm_head_argmax(_bits(fi), _bits(wi), want_logits=True)
    ref = fi.astype(np.int64) @ wi.astype(np.int64).T
    assert np.array_equal(logits, ref.astype(np.float64))
    assert np.array_equal(g, np.argmax(ref, axis=1))    # numpy also returns the first maximum
    assert not np.any(g == 17)


def test_lm_head_one_hot_feature_reads_back_a_head_column():
    rng = np.random.default_rng(5)
    H, V = 32, 77
    w = synth.normal_bf16(rng, (V, H))
    f = np.zeros((H, H), dtype=np.float32)
    f[np.arange(H), np.arange(H)] = 1.0                 # node k = unit vector e_k -> logits = head[:, k]
    g, best, logits = oracle.lm_head_argmax(_bits(f), w, want_logits=True)
    col = synth.bf16_bits_to_f32(w).astype(np.float64)
    assert np.array_equal(logits, col.T)
    assert np.array_equal(g, np.argmax(col, axis=0))


def test_lm_head_row_strides_nan_and_signed_zero():
    rng = np.random.default_rng(6)
    N, H, V = 5, 24, 31
    f = synth.normal_bf16(rng, (N, H + 8))              # junk beyond `hidden` must not be read
    w = synth.normal_bf16(rng, (V, H + 16))
    g, best = oracle.lm_head_argmax(f, w, hidden=H)
    g2, best2 = oracle.lm_head_argmax(np.ascontiguousarray(f[:, :H]), np.ascontiguousarray(w[:, :H]))
    assert np.array_equal(g, g2) and np.array_equal(best, best2)
    # a head row holding a NaN gives NaN logits, which never win; all rows NaN -> index 0
    wn = np.ascontiguousarray(w[:, :H]).copy()
    wn[int(g2[0]), 3] = 0x7FC0
    g3, _ = oracle.lm_head_argmax(np.ascontiguousarray(f[:, :H]), wn)
    assert g3[0] != g2[0]
    wn[:, 3] = 0x7FC0
    g4, _ = oracle.lm_head_argmax(np.ascontiguousarray(f[:, :H]), wn)
    assert np.all(g4 == 0)
    # -0 and +0 logits tie: features of zeros against any head -> every logit is a zero -> index 0
    z = np.zeros((2, H), dtype=np.uint16)
    z[1, :] = 0x8000
    g5, best5 = oracle.lm_head_argmax(z, np.ascontiguousarray(w[:, :H]))
    assert np.all(g5 == 0) and np.all(best5 == 0.0)


def test_lm_head_argmax_agrees_with_the_logits_scan():
    # the fused definition and "materialise fp32 logits, then oracle.argmax" pick the same token when the margin
    # between the two best logits is far above fp32 rounding
    rng = np.random.default_rng(7)
    N, H, V = 12, 128, 300
    f = synth.normal_bf16(rng, (N, H))
    w = synth.normal_bf16(rng, (V, H))
    g, best, logits = oracle.lm_head_argmax(f, w, want_logits=True)
    srt = np.sort(logits, axis=1)
    assert np.all(srt[:, -1] - srt[:, -2] > 1e-3)
    assert np.array_equal(g, oracle.argmax(np.ascontiguousarray(logits.astype(np.float32))))


# --------------------------------------------------------------------------- non-greedy token draw (Section 3.1)
def test_sample_tokens_hand_worked():
    c = GOLD["sample_tokens_basic"]
    u = np.array(c["uniform_u"], dtype=np.float32)
    lg = np.zeros((len(u), c["uniform_vocab"]), dtype=np.float32)
    assert oracle.sample_tokens(lg, 1.0, u).tolist() == c["uniform_expected"]
    assert oracle.sample_tokens(lg + 3.5, 0.7, u).tolist() == c["uniform_expected"]     # equal logits: any shift, any temperature
    ub = np.array(c["b_u"], dtype=np.float32)
    lb = np.tile(np.array(c["b_logits"], dtype=np.float32), (len(ub), 1))
    assert oracle.sample_tokens(lb, c["b_temperature"], ub).tolist() == c["b_expected"]


def test_sample_tokens_is_the_inverse_cdf_of_the_softmax():
    rng = np.random.default_rng(8)
    N, V, T = 40, 300, 1.7
    lg = (2.0 * rng.standard_normal((N, V))).astype(np.float32)
    u = rng.random(N).astype(np.float32)
    g, cdf = oracle.sample_tokens(lg, T, u, want_cdf=True)
    z = lg.astype(np.float64) / T
    p = np.exp(z - z.max(axis=1, keepdims=True))
    ref_cdf = np.cumsum(p, axis=1) / p.sum(axis=1, keepdims=True)      # numpy's softmax partial sums
    assert np.allclose(cdf, ref_cdf, rtol=1e-12, atol=1e-15)
    assert np.all(np.diff(cdf, axis=1) >= 0) and np.allclose(cdf[:, -1], 1.0)
    ref = np.array([np.searchsorted(ref_cdf[i], u[i], side="right") for i in range(N)])
    assert np.min(np.abs(ref_cdf - u[:, None].astype(np.float64))) > 1e-9   # no draw sits on a boundary
    assert np.array_equal(g, ref)
    assert np.array_equal(oracle.sample_tokens(lg + 11.0, T, u), g)    # softmax ignores a shift of the logits


def test_sample_tokens_frequencies_follow_the_probabilities():
    rng = np.random.default_rng(9)
    V, T, draws = 6, 2.0, 40000
    row = np.array([0.3, -1.0, 2.2, 0.0, 1.1, -3.0], dtype=np.float32)
    p = np.exp(row.astype(np.float64) / T)
    p /= p.sum()
    g = oracle.sample_tokens(np.tile(row, (draws, 1)), T, rng.random(draws).astype(np.float32))
    freq = np.bincount(g, minlength=V) / draws
    assert np.all(np.abs(freq - p) < 5.0 * np.sqrt(p * (1 - p) / draws))


def test_sample_tokens_limits_and_special_values():
    rng = np.random.default_rng(10)
    N, V = 25, 500
    lg = rng.standard_normal((N, V)).astype(np.float32)
    lg[np.arange(N), rng.integers(0, V, N)] += 3.0                      # a clear maximum per row
    u = rng.random(N).astype(np.float32)
    assert np.array_equal(oracle.sample_tokens(lg, 1e-3, u), oracle.argmax(lg))   # temperature -> 0: the greedy token
    one = np.full((4, 50), -np.inf, dtype=np.float32)
    one[np.arange(4), [7, 0, 49, 20]] = [1.0, -2.0, 0.5, 30.0]
    for uu in (0.0, 0.5, 0.999):                                        # a single possible token: it is drawn
        assert oracle.sample_tokens(one, 1.0, np.full(4, uu, np.float32)).tolist() == [7, 0, 49, 20]
    nan = lg.copy()
    g0 = oracle.sample_tokens(lg, 1.0, u)
    nan[np.arange(N), g0] = np.nan                                      # the drawn token becomes impossible
    g1 = oracle.sample_tokens(nan, 1.0, u)
    assert np.all(g1 != g0)
    assert np.all(oracle.sample_tokens(np.full((3, 9), np.nan, np.float32), 1.0, np.full(3, 0.4, np.float32)) == 0)
    pad = np.concatenate([lg, np.full((N, 12), 80.0, np.float32)], axis=1)   # beyond `vocab`: never read
    assert np.array_equal(oracle.sample_tokens(np.ascontiguousarray(pad), 1.0, u, vocab=V), g0)
