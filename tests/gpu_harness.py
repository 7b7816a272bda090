"""Helpers for the GPU parity tests: move seeded host inputs to the device, call
the C ABI through the binding, bring results back as numpy arrays."""
from __future__ import annotations

import math

import numpy as np
import torch

import paper_2412_12639_b200 as falcon
from paper_2412_12639_b200 import binding, synth

ATOL = 2e-2      # max |gpu - oracle| on attention outputs (bf16 kernel vs fp32 oracle)
REL_L2 = 1e-2    # per (sequence, head) block: ||gpu - oracle||_2 / ||oracle||_2

_ctx = None


def ctx() -> falcon.Context:
    global _ctx
    if _ctx is None:
        _ctx = falcon.Context(0)
    return _ctx


def dev_i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def host_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class DevTrees:
    def __init__(self, trees: synth.TreeBatch, max_prefix_len=None):
        self.host = trees
        self.node_off = dev_i32(trees.node_off)
        self.parent = dev_i32(trees.parent)
        self.token = dev_i32(trees.token)
        self.prefix_len = dev_i32(trees.prefix_len)
        self.status = torch.zeros(trees.batch, dtype=torch.int32, device="cuda")
        self.max_prefix_len = int(max(0, trees.prefix_len.max())) if max_prefix_len is None else max_prefix_len

    def desc(self, with_status=True, host_copies=False):
        t = self.host
        self._host_keep = (np.ascontiguousarray(t.prefix_len, dtype=np.int32),
                           np.ascontiguousarray(t.node_off, dtype=np.int32))
        return binding.tree_desc(t.batch, t.total_nodes, t.max_tree, self.max_prefix_len, self.node_off, self.parent,
                                 self.prefix_len, token=self.token,
                                 prefix_len_host=self._host_keep[0] if host_copies else None,
                                 node_off_host=self._host_keep[1] if host_copies else None,
                                 status=self.status if with_status else None)


def make_trees(sizes, prefs, rng, vocab=100, parents=None) -> synth.TreeBatch:
    node_off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    if parents is None:
        parents = [synth.random_shape_tree(rng, t) for t in sizes]
    parent = np.concatenate(parents).astype(np.int32)
    token = rng.integers(0, vocab, size=int(node_off[-1])).astype(np.int32)
    return synth.TreeBatch(node_off, parent, token, np.asarray(prefs, np.int32), np.full(len(sizes), 0.5))


def run_attn(dt: DevTrees, Hq, Hkv, D, q, k, v, s_cap=None, scale=None, kernel=binding.ATTN_AUTO, n_splits=0,
             k_tree=None, v_tree=None, tree_mask=None, check=True, host_copies=False, flags=0):
    """q [N,Hq,D], k/v [B,Hkv,s_cap,D] uint16 bit patterns -> (out bits [N,Hq,D], rc)."""
    scale = 1.0 / math.sqrt(D) if scale is None else scale
    qd, kd, vd = dev_bf16(q), dev_bf16(k), dev_bf16(v)
    out = torch.full_like(qd, float("nan"))
    ktd = dev_bf16(k_tree) if k_tree is not None else None
    vtd = dev_bf16(v_tree) if v_tree is not None else None
    md = torch.from_numpy(np.ascontiguousarray(tree_mask).view(np.int64)).cuda() if tree_mask is not None else None
    strides = tuple(int(s) for s in kd.stride()[:3])
    a = binding.attn_args(dt.desc(host_copies=host_copies), Hq, Hkv, D, scale, qd, out, kd, vd, strides,
                          kd.shape[2] if s_cap is None else s_cap, k_tree=ktd, v_tree=vtd, tree_mask=md,
                          kernel=kernel, n_splits=n_splits, flags=flags)
    rc = ctx().falcon_tree_attn(a, check=check)
    torch.cuda.synchronize()
    return host_bits(out), rc


ROW_REL_L2 = 1e-2  # per (node, head) row: ||gpu - oracle||_2 / max(||oracle||_2, ROW_FLOOR)
ROW_FLOOR = 0.05   # rows whose oracle norm is below this are measured against it (a near-zero row has no scale of its own)
RTOL = 1e-2        # elementwise |gpu - oracle| <= ATOL + RTOL * |oracle|


def attn_errors(out_bits, ref, node_off):
    """max abs error, the worst per-(sequence, head) relative L2 error, the worst per-(node, head) row relative L2
    error (with its node and head) and the fraction of elements inside |d| <= ATOL + RTOL * |ref|."""
    got = synth.bf16_bits_to_f32(out_bits).astype(np.float64)
    ref = ref.astype(np.float64)
    assert np.isfinite(got).all(), "non-finite attention output"
    d = got - ref
    max_abs = float(np.abs(d).max())
    worst = 0.0
    for b in range(len(node_off) - 1):
        lo, hi = node_off[b], node_off[b + 1]
        num = np.sqrt((d[lo:hi] ** 2).sum(axis=(0, 2)))
        den = np.sqrt((ref[lo:hi] ** 2).sum(axis=(0, 2)))
        worst = max(worst, float((num / np.maximum(den, 1e-30)).max()))
    row = np.sqrt((d ** 2).sum(axis=2)) / np.maximum(np.sqrt((ref ** 2).sum(axis=2)), ROW_FLOOR)
    at = np.unravel_index(int(np.argmax(row)), row.shape)
    inside = float((np.abs(d) <= ATOL + RTOL * np.abs(ref)).mean())
    return max_abs, worst, float(row[at]), (int(at[0]), int(at[1])), inside


def assert_attn_close(out_bits, ref, node_off, report=False):
    max_abs, rel, row_rel, row_at, inside = attn_errors(out_bits, ref, node_off)
    if report:
        print("attention vs oracle: max abs %.3g, block rel L2 %.3g, worst row rel L2 %.3g at (node %d, head %d), "
              "allclose(atol %.0e, rtol %.0e) fraction %.6f" % (max_abs, rel, row_rel, row_at[0], row_at[1], ATOL, RTOL, inside))
    assert max_abs <= ATOL, "max abs error %.4g > %.4g" % (max_abs, ATOL)
    assert rel <= REL_L2, "relative L2 error %.4g > %.4g" % (rel, REL_L2)
    assert row_rel <= ROW_REL_L2, "row (node %d, head %d): relative L2 error %.4g > %.4g" % (row_at + (row_rel, ROW_REL_L2))
    assert inside == 1.0, "elements outside atol + rtol * |ref|: fraction %.3g" % (1.0 - inside)
    return max_abs, rel


def run_accept(dt: DevTrees, logits: np.ndarray, vocab=None, path_stride=128, temperature=0.0, uniforms=None):
    """logits fp32 [N, stride] -> (g, path, n_path, next_token) numpy.  temperature > 0: the non-greedy call
    with uniforms fp32 [N]."""
    ld = torch.from_numpy(np.ascontiguousarray(logits)).cuda()
    ud = None if uniforms is None else torch.from_numpy(np.ascontiguousarray(uniforms, dtype=np.float32)).cuda()
    N, B = dt.host.total_nodes, dt.host.batch
    g = torch.full((N,), -7, dtype=torch.int32, device="cuda")
    path = torch.full((B, path_stride), -7, dtype=torch.int32, device="cuda")
    n_path = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    nxt = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    a = binding.accept_args(dt.desc(), logits.shape[1] if vocab is None else vocab, ld, logits.shape[1], g, path,
                            path_stride, n_path, nxt, temperature=temperature, uniforms=ud)
    ctx().falcon_tree_accept(a)
    torch.cuda.synchronize()
    return g.cpu().numpy(), path.cpu().numpy(), n_path.cpu().numpy(), nxt.cpu().numpy()


def run_topm(logits: np.ndarray, m, vocab=None, check=True):
    """logits fp32 [N, stride] -> (values [N, m], indices [N, m], rc)."""
    ld = torch.from_numpy(np.ascontiguousarray(logits)).cuda()
    N, stride = ld.shape
    V = stride if vocab is None else vocab
    val = torch.full((N, m), float("nan"), dtype=torch.float32, device="cuda")
    idx = torch.full((N, m), -7, dtype=torch.int32, device="cuda")
    rc = ctx().falcon_topm(binding.topm_args(N, V, ld, stride, m, val, idx), check=check)
    torch.cuda.synchronize()
    return val.cpu().numpy(), idx.cpu().numpy(), rc


def run_compact(dt: DevTrees, Hkv, D, k_layers, v_layers, path, n_path, k_tree_layers=None, v_tree_layers=None,
                s_cap=None):
    """k_layers / v_layers: lists of uint16 [B,Hkv,s_cap,D] host arrays.  Returns compacted copies and new_len."""
    kd = [dev_bf16(x) for x in k_layers]
    vd = [dev_bf16(x) for x in v_layers]
    kp = torch.tensor([t.data_ptr() for t in kd], dtype=torch.int64, device="cuda")
    vp = torch.tensor([t.data_ptr() for t in vd], dtype=torch.int64, device="cuda")
    ktd = vtd = ktp = vtp = None
    if k_tree_layers is not None:
        ktd = [dev_bf16(x) for x in k_tree_layers]
        vtd = [dev_bf16(x) for x in v_tree_layers]
        ktp = torch.tensor([t.data_ptr() for t in ktd], dtype=torch.int64, device="cuda")
        vtp = torch.tensor([t.data_ptr() for t in vtd], dtype=torch.int64, device="cuda")
    pd, nd = dev_i32(path), dev_i32(n_path)
    new_len = torch.full((dt.host.batch,), -7, dtype=torch.int32, device="cuda")
    strides = tuple(int(s) for s in kd[0].stride()[:3])
    a = binding.compact_args(dt.desc(), len(kd), Hkv, D, kp, vp, strides, kd[0].shape[2] if s_cap is None else s_cap,
                             pd, pd.shape[1], nd, new_len, k_tree_layers=ktp, v_tree_layers=vtp)
    ctx().falcon_kv_compact(a)
    torch.cuda.synchronize()
    return [host_bits(t) for t in kd], [host_bits(t) for t in vd], new_len.cpu().numpy()


def run_lm_argmax(feat_bits, head_bits, hidden=None, check=True):
    """falcon_lm_head_argmax on uint16 bf16 bit patterns [N, feat_stride] / [V, head_stride].
    Returns (argmax [N], max [N] fp32, status word, rc)."""
    N, fs = feat_bits.shape
    V, hs = head_bits.shape
    Hd = min(fs, hs) if hidden is None else hidden
    f, w = dev_bf16(feat_bits), dev_bf16(head_bits)
    g = torch.full((N,), -3, dtype=torch.int32, device="cuda")
    mx = torch.full((N,), -7.0, dtype=torch.float32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    rc = ctx().falcon_lm_head_argmax(binding.lm_argmax_args(N, Hd, V, f, fs, w, hs, g, mx, st), check=check)
    torch.cuda.synchronize()
    return g.cpu().numpy(), mx.cpu().numpy(), int(st.item()), rc
