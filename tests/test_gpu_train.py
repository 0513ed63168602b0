"""Training-time attention (Section 3.2 "Training"): forward and backward of the layers before the split (every token,
ordinary causal attention) and after it (registers and target tokens only), against the oracle."""
import numpy as np
import pytest
import torch

from oracle import earn_oracle as orc
from paper_2507_00715_b200 import binding as B
from paper_2507_00715_b200 import workloads as wl
from parity_util import TOL, to_np

pytestmark = pytest.mark.gpu


def _close(got: torch.Tensor, ref: np.ndarray, dtype: str, what: str, scale: float = 1.0):
    """Gradients are sums over up to L terms of O(1) products: their bound scales with their own magnitude
    (`scale` = the largest reference value, at least 1), the relative precision being that of one bf16 rounding."""
    g = got.detach().double().cpu().numpy()
    assert g.shape == ref.shape, (what, g.shape, ref.shape)
    if g.size == 0:
        return
    assert np.isfinite(g).all(), what
    err = np.abs(g - ref)
    t = TOL[dtype]
    assert err.max() <= t["max_abs"] * scale, f"{what}: max abs err {err.max():.3e} (bound {t['max_abs'] * scale:.3e})"
    assert err.mean() <= t["mean_abs"] * scale, f"{what}: mean abs err {err.mean():.3e}"


def _setup(w, n_target):
    model = B.make_model(w.n_layers, w.split_k, w.n_q_heads, w.n_kv_heads, w.head_dim, w.torch_dtype)
    batch = B.Batch(wl.cu_seqlens(w), w.r_head, w.r_tail)
    ws = torch.empty(B.earn_train_workspace_bytes(model, batch), dtype=torch.uint8, device="cuda")
    B.earn_workspace_init(ws)
    return model, batch, ws


def run_full_layer(w, n_target=4, sample_seqs=None):
    """A layer before the split: every token attends causally.  Compared in full, or on whole sampled sequences."""
    model, batch, ws = _setup(w, n_target)
    cu = wl.cu_seqlens(w)
    total = int(cu[-1])
    q, k, v = wl.layer_qkv(w, 0, "cuda")
    d_o = wl.upstream_grad(w, 0, q.shape, "cuda")
    o = torch.empty_like(q)
    lse = torch.empty(w.n_q_heads, total, dtype=torch.float32, device="cuda")
    dq, dk, dv = torch.full_like(q, float("nan")), torch.full_like(k, float("nan")), torch.full_like(v, float("nan"))
    B.earn_train_attn_fwd(model, batch, 0, n_target, q, k, v, o, lse, ws)
    B.earn_train_attn_bwd(model, batch, 0, n_target, q, k, v, o, lse, d_o, dq, dk, dv, ws)
    torch.cuda.synchronize()
    assert B.earn_device_status(ws) == 0
    seqs = range(w.batch) if sample_seqs is None else sample_seqs
    for b in seqs:
        sl = slice(int(cu[b]), int(cu[b + 1]))
        qn, kn, vn, gn = to_np(q[sl]), to_np(k[sl]), to_np(v[sl]), to_np(d_o[sl])
        c1 = np.array([0, sl.stop - sl.start])
        o_ref, lse_ref = orc.causal_attention(qn, kn, vn, c1)
        _close(o[sl], o_ref, w.dtype, f"O seq {b}")
        assert np.abs(lse[:, sl].double().cpu().numpy() - lse_ref).max() <= (1e-4 if w.dtype == "f32" else 2e-2)
        dq_ref, dk_ref, dv_ref = orc.causal_attention_grad(qn, kn, vn, c1, gn)
        for name, got, ref in (("dQ", dq[sl], dq_ref), ("dK", dk[sl], dk_ref), ("dV", dv[sl], dv_ref)):
            _close(got, ref, w.dtype, f"{name} seq {b}", scale=max(1.0, float(np.abs(ref).max())))
    return dq, dk, dv


def run_participating_layer(w, n_target=4):
    """A layer after the split: the gathered rows [prefix; suffix; targets] of every sequence, causal among themselves."""
    model, batch, ws = _setup(w, n_target)
    cu, lens = wl.cu_seqlens(w), wl.seqlens(w)
    idx = orc.participating_indices(lens, w.r_head, w.r_tail, n_target)
    P = idx.shape[1]
    layer = w.split_k
    qf, kf, vf = wl.layer_qkv(w, layer, "cuda")
    rows = torch.from_numpy((cu[:-1, None] + idx).astype(np.int64)).cuda()          # the gather X -> X' of Section 3.2
    q, k, v = qf[rows].contiguous(), kf[rows].contiguous(), vf[rows].contiguous()   # [B, P, H, D]
    d_o = wl.upstream_grad(w, layer, q.shape, "cuda")
    o = torch.empty_like(q)
    lse = torch.empty(w.batch, w.n_q_heads, P, dtype=torch.float32, device="cuda")
    dq, dk, dv = torch.full_like(q, float("nan")), torch.full_like(k, float("nan")), torch.full_like(v, float("nan"))
    B.earn_train_attn_fwd(model, batch, layer, n_target, q, k, v, o, lse, ws)
    B.earn_train_attn_bwd(model, batch, layer, n_target, q, k, v, o, lse, d_o, dq, dk, dv, ws)
    torch.cuda.synchronize()
    qn, kn, vn = to_np(qf), to_np(kf), to_np(vf)
    q_p, k_p, v_p = orc.compact(qn, cu, idx), orc.compact(kn, cu, idx), orc.compact(vn, cu, idx)
    o_ref, lse_ref = orc.participating_attention(q_p, k_p, v_p)
    _close(o, o_ref, w.dtype, "O'")
    if P > 0:
        assert np.abs(lse.double().cpu().numpy() - lse_ref).max() <= (1e-4 if w.dtype == "f32" else 2e-2)
    dq_ref, dk_ref, dv_ref = orc.participating_attention_grad(q_p, k_p, v_p, to_np(d_o))
    for name, got, ref in (("dQ'", dq, dq_ref), ("dK'", dk, dk_ref), ("dV'", dv, dv_ref)):
        _close(got, ref, w.dtype, name, scale=max(1.0, float(np.abs(ref).max())) if ref.size else 1.0)


TINY = wl.CONFIGS["tiny"]
SMALL = wl.Workload("train", batch=3, n_layers=2, split_k=1, n_q_heads=8, n_kv_heads=2, head_dim=128, dtype="bf16",
                    prompt_len=0, lens=(200, 77, 333), r_head=5, r_tail=3, seed=51)


def test_tiny_fp32_both_sides_of_the_split():
    run_full_layer(TINY)
    run_participating_layer(TINY)


@pytest.mark.parametrize("kw", [dict(), dict(n_q_heads=6, n_kv_heads=2), dict(n_q_heads=2, n_kv_heads=2, lens=(128, 129, 1, 260), batch=4, r_head=0, r_tail=0, n_target=1),
                                dict(head_dim=64), dict(dtype="f32", lens=(65, 140), batch=2)])
def test_full_layers_small_ragged(kw):
    kw = dict(kw)
    n_target = kw.pop("n_target", 4)
    run_full_layer(SMALL.replace(**kw), n_target=n_target)


@pytest.mark.parametrize("rh,rt,nt", [(5, 3, 4), (0, 2, 4), (16, 16, 4), (1, 1, 0), (0, 0, 3), (0, 0, 0), (30, 30, 8)])
def test_participating_layers(rh, rt, nt):
    run_participating_layer(SMALL.replace(r_head=rh, r_tail=rt), n_target=nt)
    run_participating_layer(SMALL.replace(r_head=rh, r_tail=rt, dtype="f32", head_dim=64, n_q_heads=4), n_target=nt)


def test_full_layer_7b_shapes_sampled_sequences():
    """The measured shape (64 sequences of 1024 tokens, 32 query heads over 8 kv heads): O, LSE, dQ, dK, dV of two whole
    sequences (the first and the last) against the oracle; eight key tiles per sequence, groups of four heads adding
    into each kv head, 36 (query tile, key tile) pairs per head."""
    run_full_layer(wl.CONFIGS["7b"].replace(n_layers=2, split_k=1, decode_steps=0), sample_seqs=(0, 63))


def test_full_layer_long_and_ragged_sampled_sequences():
    w = wl.CONFIGS["ragged"].replace(n_layers=2, split_k=1, decode_steps=0, beams=1, batch=24)
    lens = wl.seqlens(w)
    run_full_layer(w, sample_seqs=(int(np.argmin(lens)), int(np.argmax(lens)), 23))


def test_backward_is_reproducible():
    w = SMALL.replace(seed=52)
    a = run_full_layer(w)
    b = run_full_layer(w)
    for x, y in zip(a, b):
        assert torch.equal(x, y)
