"""Hidden-state form of the register layers (Section 3.2, register-focused process; Eq. 2 on X'): the CUDA projection
(gather, RMSNorm, tcgen05 GEMM, rotary embedding, paged cache write) against the oracle, element by element."""
import numpy as np
import pytest
import torch

from oracle import earn_oracle as orc
from paper_2507_00715_b200 import binding as B
from paper_2507_00715_b200 import workloads as wl
from parity_util import assert_close, make_session, to_np

pytestmark = pytest.mark.gpu


def _base(**kw):
    d = dict(name="regqkv", batch=3, n_layers=3, split_k=1, n_q_heads=4, n_kv_heads=2, head_dim=128, dtype="bf16",
             prompt_len=0, lens=(40, 17, 300), r_head=4, r_tail=4, seed=21, hidden=512)
    d.update(kw)
    return wl.Workload(**d)


def _cache_rows(ses, t, seqs, R):
    """Rows 0..R-1 of the given sequences' compact cache, read through the page table: [len(seqs), R, Hkv, D]."""
    nb = ses.batch.batch
    pages = (ses.block_table.cpu().numpy() if ses.block_table is not None
             else np.arange(ses.n_pages).reshape(nb, ses.pages_per_seq))
    a = to_np(t)
    return np.stack([np.stack([a[pages[b, m // 16], m % 16] for m in range(R)]) for b in seqs])


def _oracle_rows(w, x, wn, wq, cu, idx, cos, sin, seqs, compact):
    """Q', K', V' of the chosen sequences from the oracle, one sequence per call."""
    R = w.n_regs
    out = ([], [], [])
    for b in seqs:
        if compact:
            # x holds the register rows alone: a "sequence" of R rows, row m rotated by its original position idx[b][m]
            # (the oracle indexes the tables by the row it gathers, so hand it the table rows of those positions)
            got = orc.register_qkv(x[b * R:(b + 1) * R], np.array([0]), np.arange(R)[None], wn, wq, w.n_q_heads,
                                   w.n_kv_heads, w.head_dim, cos[idx[b]], sin[idx[b]])
        else:
            got = orc.register_qkv(x[cu[b]:cu[b + 1]], np.array([0]), idx[b:b + 1], wn, wq, w.n_q_heads, w.n_kv_heads,
                                   w.head_dim, cos, sin)
        for dst, g in zip(out, got):
            dst.append(g[0])
    return tuple(np.stack(t) for t in out)


def _run(w, compact=False, layers=None, sample=None, **session_kw):
    cu, lens = wl.cu_seqlens(w), wl.seqlens(w)
    idx = orc.register_indices(lens, w.r_head, w.r_tail)
    max_pos = int(lens.max())
    ses = make_session(w, **session_kw)
    ses.set_projection(w.d_model, max_pos)
    cos, sin = orc.rope_tables(max_pos, w.head_dim)
    R = w.n_regs
    seqs = list(range(w.batch)) if sample is None else list(sample)
    for layer in (layers if layers is not None else range(w.split_k, w.n_layers)):
        x = wl.hidden_states(w, layer, "cuda", compact=compact)
        wn, wq = wl.projection_weights(w, layer, "cuda")
        o = ses.register_layer_from_hidden(layer, x, wn, wq, x_is_compact=compact)
        assert ses.device_status() == B.EARN_OK
        q_ref, k_ref, v_ref = _oracle_rows(w, to_np(x), to_np(wn), to_np(wq), cu, idx, cos, sin, seqs, compact)
        assert np.array_equal(ses.reg_idx.cpu().numpy()[:, :R], idx)
        assert_close(ses.last_q_reg[seqs], q_ref, "bf16", f"Q' layer {layer}")
        assert_close(torch.from_numpy(_cache_rows(ses, ses.k_shared[layer], seqs, R)), k_ref, "bf16", f"K' layer {layer}")
        assert_close(torch.from_numpy(_cache_rows(ses, ses.v_shared[layer], seqs, R)), v_ref, "bf16", f"V' layer {layer}")
        # The attention call that follows is checked on its own: the oracle gets the Q', K', V' that the projection
        # STORED (read back from q_reg and the cache pages), so the bound below is the bound of one attention call.
        q_st = ses.last_q_reg[seqs].double().cpu().numpy()
        k_st = _cache_rows(ses, ses.k_shared[layer], seqs, R).astype(np.float64)
        v_st = _cache_rows(ses, ses.v_shared[layer], seqs, R).astype(np.float64)
        assert_close(o[seqs], orc.register_attention(q_st, k_st, v_st), "bf16", f"register attention layer {layer}")
    return ses


def test_small_ragged_one_tile():
    """24 register rows (one ragged row tile), 8 heads, 8 k-blocks; few tiles, so one head per tile."""
    _run(_base())


def test_scattered_pages_and_odd_head_count():
    """Hq + 2 Hkv = 5 heads: the last 256-column tile is half outside W_qkv; pages scattered through a block table."""
    _run(_base(n_q_heads=3, n_kv_heads=1, r_head=9, r_tail=10, lens=(64, 19, 130, 77), batch=4, hidden=256),
         paged_shuffle_seed=5)


def test_compact_hidden_states():
    """x already holds only the register rows (every register layer after the first)."""
    _run(_base(), compact=True)


def test_several_tiles_per_cta():
    """1280 rows x 64 heads = 320 output tiles: every CTA takes two or three, so both accumulators and the ring wrap."""
    w = _base(batch=40, lens=(), prompt_len=0, len_lo=40, len_hi=400, r_head=16, r_tail=16, n_q_heads=56, n_kv_heads=4,
              hidden=256, n_layers=2, seed=22)
    _run(w, sample=(0, 7, 39))


def test_two_head_tiles_with_an_odd_head_count():
    """1280 rows x 21 heads: enough tiles for the two-heads-per-tile kernel, whose last tile is half outside W_qkv."""
    w = _base(batch=40, lens=(), prompt_len=0, len_lo=40, len_hi=400, r_head=16, r_tail=16, n_q_heads=15, n_kv_heads=3,
              hidden=256, n_layers=2, seed=24)
    _run(w, sample=(1, 20, 38))


def test_deep_k():
    """d_model 2048: 32 k-blocks per tile, the 4-stage ring wraps eight times; two row tiles, ragged."""
    w = _base(batch=5, lens=(100, 64, 333, 32, 50), r_head=16, r_tail=16, n_q_heads=8, n_kv_heads=2, hidden=2048,
              n_layers=2, seed=23)
    _run(w)


def test_no_registers_is_a_no_op():
    w = _base(r_head=0, r_tail=0)
    ses = make_session(w)
    ses.set_projection(w.d_model, 512)
    x = wl.hidden_states(w, 1, "cuda")
    wn, wq = wl.projection_weights(w, 1, "cuda")
    n0 = B.earn_launch_count()
    q_reg = torch.empty(w.batch, 0, w.n_q_heads, w.head_dim, device="cuda", dtype=torch.bfloat16)
    B.earn_register_qkv(ses.model, ses.batch, 1, B.make_proj(w.d_model, ses.rope_cos, ses.rope_sin), x, wn, wq, ses.x_norm,
                        ses.cache(1), q_reg, ses.workspace)
    assert B.earn_launch_count() == n0


def test_rejects_bad_arguments():
    w = _base()
    ses = make_session(w)
    ses.set_projection(w.d_model, 512)
    x = wl.hidden_states(w, 1, "cuda")
    wn, wq = wl.projection_weights(w, 1, "cuda")
    q_reg = torch.empty(w.batch, w.n_regs, w.n_q_heads, w.head_dim, device="cuda", dtype=torch.bfloat16)
    args = lambda proj, layer=1: (ses.model, ses.batch, layer, proj, x, wn, wq, ses.x_norm, ses.cache(1), q_reg, ses.workspace)
    good = B.make_proj(w.d_model, ses.rope_cos, ses.rope_sin)
    with pytest.raises(B.EarnError):   # layer below the split
        B.earn_register_qkv(*args(good, layer=0))
    with pytest.raises(B.EarnError):   # d_model not a multiple of 64
        B.earn_register_qkv(*args(B.make_proj(w.d_model + 8, ses.rope_cos, ses.rope_sin)))
    with pytest.raises(B.EarnError):   # a prompt longer than the rotary tables
        B.earn_register_qkv(*args(B.make_proj(w.d_model, ses.rope_cos[:100], ses.rope_sin[:100])))
    B.earn_register_qkv(*args(good))
    assert ses.device_status() == B.EARN_OK


def test_full_size_7b_layer_sampled_sequences():
    """The measured shape (64 prompts of 1024 tokens, 32 registers, d_model 4096, 48 heads of W_qkv): 2048 x 6144 x 4096,
    384 output tiles; three sequences' rows (the first, one inside, the last) compared element by element."""
    w = wl.CONFIGS["7b"].replace(n_layers=9, split_k=8, decode_steps=0)
    _run(w, sample=(0, 31, 63))
