"""falcon_tree_accept_static: the acceptance call for hosts that are not allowed
to allocate device memory (a server whose memory pool owns the whole GPU, a
process on a fixed memory budget, a loop that must never hit an allocation's
synchronisation).  Its scratch is a fixed array inside the library, so the
test checks these things through the C ABI: it returns exactly what
falcon_tree_accept and the CPU oracle return, it still does so on a second call
in a row (the array keeps the first call's contents), the free device memory
does not move between its first call and its tenth (the one property the call
exists for), and sizes beyond the fixed array are refused instead of being
served partially.

This file is collected last on purpose: a run that stops at the first failure
has then already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2412_12639_b200 import binding, synth

import gpu_harness as H

pytestmark = pytest.mark.gpu


def run_static(dt, logits_dev, vocab, stride):
    N, B = dt.host.total_nodes, dt.host.batch
    g = torch.full((N,), -7, dtype=torch.int32, device="cuda")
    path = torch.full((B, 128), -7, dtype=torch.int32, device="cuda")
    n_path = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    nxt = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    a = binding.accept_args(dt.desc(), vocab, logits_dev, stride, g, path, 128, n_path, nxt)
    binding.falcon_tree_accept_static(a)
    torch.cuda.synchronize()
    return g.cpu().numpy(), path.cpu().numpy(), n_path.cpu().numpy(), nxt.cpu().numpy()


@pytest.mark.parametrize("name", ["v7b", "ragged"])
def test_static_accept_matches_the_allocating_entry_point_twice_in_a_row(name):
    spec = synth.SPECS[name]
    tb = synth.make_trees(spec)
    logits = synth.make_logits(spec, tb)
    dt = H.DevTrees(tb)
    want = H.run_accept(dt, logits)                       # existing entry point (context scratch)
    g_ref = oracle.argmax(logits)                         # and the CPU oracle, directly
    p_ref, n_ref, t_ref = oracle.tree_accept(tb.node_off, tb.parent, tb.token, g_ref)
    ld = torch.from_numpy(logits).cuda()
    for _ in range(2):                                    # second call reuses the array as the first left it
        got = run_static(dt, ld, spec.vocab, logits.shape[1])
        for w, g_ in zip(want, got):
            np.testing.assert_array_equal(g_, w)          # integer results: bit-exact
        for w, g_ in zip((g_ref, p_ref, n_ref, t_ref), got):
            np.testing.assert_array_equal(g_, w)
    # a different, smaller problem right after: stale partials of the larger one must not leak in
    rng = np.random.default_rng(1)
    tb2 = H.make_trees([9, 33, 1], [0, 0, 0], rng, vocab=7)
    lg2 = rng.standard_normal((tb2.total_nodes, 7)).astype(np.float32)
    dt2 = H.DevTrees(tb2)
    want2 = H.run_accept(dt2, lg2)
    got2 = run_static(dt2, torch.from_numpy(lg2).cuda(), 7, 7)
    for w, g_ in zip(want2, got2):
        np.testing.assert_array_equal(g_, w)


def test_static_accept_leaves_free_device_memory_where_it_was():
    """The call allocates nothing: after its first call (which only looks up the array's address) the driver reports
    the same free memory before the second call and after the tenth, outputs and inputs being allocated beforehand."""
    spec = synth.SPECS["v7b"]
    tb = synth.make_trees(spec)
    logits = synth.make_logits(spec, tb)
    dt = H.DevTrees(tb)
    ld = torch.from_numpy(logits).cuda()
    N, B = tb.total_nodes, tb.batch
    i32 = lambda *s: torch.full(s, -7, dtype=torch.int32, device="cuda")
    g, path, n_path, nxt = i32(N), i32(B, 128), i32(B), i32(B)
    a = binding.accept_args(dt.desc(), spec.vocab, ld, logits.shape[1], g, path, 128, n_path, nxt)
    binding.falcon_tree_accept_static(a)                  # first call on this device: one-time set-up
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for _ in range(9):
        binding.falcon_tree_accept_static(a)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    g_ref = oracle.argmax(logits)
    np.testing.assert_array_equal(g.cpu().numpy(), g_ref)
    np.testing.assert_array_equal(n_path.cpu().numpy(), oracle.tree_accept(tb.node_off, tb.parent, tb.token, g_ref)[1])


def test_static_accept_refuses_sizes_beyond_its_fixed_scratch():
    rng = np.random.default_rng(2)
    sizes = [128] * 9                                     # 1152 nodes > STATIC_MAX_NODES
    tb = H.make_trees(sizes, [0] * 9, rng, vocab=5)
    assert tb.total_nodes > binding.STATIC_MAX_NODES
    dt = H.DevTrees(tb)
    lg = torch.zeros((tb.total_nodes, 8), device="cuda")
    i32 = lambda *s: torch.full(s, -7, dtype=torch.int32, device="cuda")
    g, path, n_path, nxt = i32(tb.total_nodes), i32(9, 128), i32(9), i32(9)
    a = binding.accept_args(dt.desc(), 8, lg, 8, g, path, 128, n_path, nxt)
    assert binding.falcon_tree_accept_static(a, check=False) == binding.ERR_CAPACITY
    torch.cuda.synchronize()
    assert (n_path.cpu().numpy() == -7).all()             # nothing was launched
    with pytest.raises(binding.FalconError):
        binding.falcon_tree_accept_static(a)
