"""Parity at the full sizes of the measured workloads, in the launch configuration the benchmark times.

The oracle cannot compute these workloads in full, so the attention outputs are compared on sampled rows it
computes one by one (first and last rows of sequences, rows on either side of every 128-row tile edge of the
sampled sequences, the shortest and the longest sequence, random rows), while compaction (index list, cache
pages, gathered queries) is compared in full, bit for bit.  One full layer and one register layer per workload:
the kernels and their grids depend on the batch shape, not on how many layers repeat them.
"""
import numpy as np
import pytest
import torch

from oracle import earn_oracle as orc
from paper_2507_00715_b200 import workloads as wl
from parity_util import TOL, make_session, to_np

pytestmark = pytest.mark.gpu


def sampled_prefill_rows(w, cu, rng, n_random):
    lens = np.diff(cu)
    seqs = {0, w.batch - 1, int(np.argmin(lens)), int(np.argmax(lens))}
    seqs |= set(int(b) for b in rng.integers(0, w.batch, size=3))
    toks = set()
    for b in seqs:
        L = int(lens[b])
        cand = {0, 1, L - 1, L - 2, w.r_head, L - w.r_tail - 1, L - w.r_tail}
        for edge in range(128, L, 128):
            cand |= {edge - 1, edge, edge + 1}
        toks |= {int(cu[b]) + t for t in cand if 0 <= t < L}
    tok = np.array(sorted(toks), dtype=np.int64)
    head = rng.integers(0, w.n_q_heads, size=len(tok))
    # every head of one kv group on a few of those rows (the heads of a group share K/V tiles in one CTA)
    extra_t = np.repeat(tok[:: max(1, len(tok) // 8)], w.group)
    extra_h = np.tile(np.arange(w.group), len(extra_t) // w.group) + w.group * int(rng.integers(0, w.n_kv_heads))
    rt = rng.integers(0, int(cu[-1]), size=n_random)
    rh = rng.integers(0, w.n_q_heads, size=n_random)
    return np.concatenate([tok, extra_t, rt]), np.concatenate([head, extra_h, rh])


def check(got, ref, dtype, what):
    err = np.abs(got - ref)
    t = TOL[dtype]
    assert np.isfinite(got).all(), what
    assert err.max() <= t["max_abs"], f"{what}: max abs err {err.max():.3e}"
    assert err.mean() <= t["mean_abs"], f"{what}: mean abs err {err.mean():.3e}"


def run_fullsize(w, decode_steps=2, n_random=1500, n_decode_rows=600):
    w = w.replace(n_layers=2, split_k=1, decode_steps=decode_steps)
    rng = np.random.Generator(np.random.Philox(w.seed + 77))
    cu = wl.cu_seqlens(w)
    lens = wl.seqlens(w)
    ses = make_session(w)
    idx = orc.register_indices(lens, w.r_head, w.r_tail)

    # ---- layer 0: full causal prefill, sampled rows
    q, k, v = wl.layer_qkv(w, 0, "cuda")
    o = ses.prefill_layer(0, q, k, v)
    o2 = ses.prefill_layer(0, q, k, v, out=torch.empty_like(o))
    assert torch.equal(o, o2), "prefill is not reproducible from launch to launch"
    qn, kn, vn = to_np(q), to_np(k), to_np(v)
    tok, head = sampled_prefill_rows(w, cu, rng, n_random)
    ref = orc.causal_attention_rows(qn, kn, vn, cu, tok, head)
    got = o[torch.from_numpy(tok).cuda(), torch.from_numpy(head).cuda()].double().cpu().numpy()
    check(got, ref, w.dtype, f"{w.name} prefill, {len(tok)} sampled rows")
    full_k = [kn[cu[b]:cu[b + 1]] for b in range(w.batch)]
    full_v = [vn[cu[b]:cu[b + 1]] for b in range(w.batch)]
    del qn

    # ---- layer 1: compaction in full (bit-exact), register attention in full
    q1, k1, v1 = wl.layer_qkv(w, 1, "cuda")
    o_reg = ses.prefill_layer(1, q1, k1, v1)
    q1n, k1n, v1n = to_np(q1), to_np(k1), to_np(v1)
    kc, vc, qc = orc.compact(k1n, cu, idx), orc.compact(v1n, cu, idx), orc.compact(q1n, cu, idx)
    R = w.n_regs
    assert np.array_equal(ses.reg_idx.cpu().numpy()[:, :R], idx)
    ks = to_np(ses.k_shared[1]).reshape(w.batch, ses.pages_per_seq * 16, w.n_kv_heads, w.head_dim)[:, :R]
    vs = to_np(ses.v_shared[1]).reshape(w.batch, ses.pages_per_seq * 16, w.n_kv_heads, w.head_dim)[:, :R]
    assert ks.tobytes() == kc.tobytes() and vs.tobytes() == vc.tobytes(), "compact cache differs from the oracle"
    assert to_np(ses.last_q_reg).tobytes() == qc.tobytes()
    check(o_reg.double().cpu().numpy(), orc.register_attention(qc, kc, vc), w.dtype, f"{w.name} register attention")
    del q1n, k1n, v1n

    # ---- decode: both layers, sampled (beam, head) rows
    states = [orc.DecodeState(full_k, full_v, w.beams), orc.DecodeState(list(kc), list(vc), w.beams)]
    n_beams = w.batch * w.beams
    for step in range(1, decode_steps + 1):
        parents = wl.beam_parents(w, step) if w.beams > 1 and step > 1 else None
        ses.begin_step(step, None if parents is None else torch.from_numpy(parents).cuda())
        pick_j = np.concatenate([[0, n_beams - 1], rng.integers(0, n_beams, size=n_decode_rows)])
        pick_h = np.concatenate([[0, w.n_q_heads - 1], rng.integers(0, w.n_q_heads, size=n_decode_rows)])
        rows = set(zip(pick_j.tolist(), pick_h.tolist()))
        for layer in range(2):
            dq, dk, dv = wl.decode_qkv(w, layer, step, "cuda")
            od = ses.decode_layer(layer, step, dq, dk, dv)
            ref = states[layer].step(to_np(dq), to_np(dk), to_np(dv), parents, rows=rows)
            jj = np.array([r[0] for r in rows])
            hh = np.array([r[1] for r in rows])
            got = od.double().cpu().numpy()[jj, hh]
            check(got, ref[jj, hh], w.dtype, f"{w.name} decode step {step} layer {layer}")
    assert ses.device_status() == 0


def run_layer_mix(w, n_random=300, n_decode_rows=80, decode_steps=2):
    """Any number of layers on either side of the split: sampled prefill rows for the full layers, compaction in full and
    register attention in full for the register layers, sampled decode rows for every layer."""
    rng = np.random.Generator(np.random.Philox(w.seed + 1000 * w.split_k))
    w = w.replace(decode_steps=decode_steps)
    cu, lens = wl.cu_seqlens(w), wl.seqlens(w)
    ses = make_session(w)
    idx = orc.register_indices(lens, w.r_head, w.r_tail)
    R = w.n_regs
    states = []
    for layer in range(w.n_layers):
        q, k, v = wl.layer_qkv(w, layer, "cuda")
        o = ses.prefill_layer(layer, q, k, v)
        qn, kn, vn = to_np(q), to_np(k), to_np(v)
        if layer < w.split_k:
            tok, head = sampled_prefill_rows(w, cu, rng, n_random)
            ref = orc.causal_attention_rows(qn, kn, vn, cu, tok, head)
            got = o[torch.from_numpy(tok).cuda(), torch.from_numpy(head).cuda()].double().cpu().numpy()
            check(got, ref, w.dtype, f"{w.name} k={w.split_k} prefill layer {layer}")
            states.append(orc.DecodeState([kn[cu[b]:cu[b + 1]] for b in range(w.batch)],
                                          [vn[cu[b]:cu[b + 1]] for b in range(w.batch)], w.beams))
        else:
            kc, vc, qc = orc.compact(kn, cu, idx), orc.compact(vn, cu, idx), orc.compact(qn, cu, idx)
            assert np.array_equal(ses.reg_idx.cpu().numpy()[:, :R], idx)
            ks = to_np(ses.k_shared[layer]).reshape(w.batch, ses.pages_per_seq * 16, w.n_kv_heads, w.head_dim)[:, :R]
            vs = to_np(ses.v_shared[layer]).reshape(w.batch, ses.pages_per_seq * 16, w.n_kv_heads, w.head_dim)[:, :R]
            assert ks.tobytes() == kc.tobytes() and vs.tobytes() == vc.tobytes(), f"compact cache, layer {layer}"
            check(o.double().cpu().numpy(), orc.register_attention(qc, kc, vc), w.dtype,
                  f"{w.name} k={w.split_k} register layer {layer}")
            states.append(orc.DecodeState(list(kc), list(vc), w.beams))
    n_beams = w.batch * w.beams
    for step in range(1, decode_steps + 1):
        pick_j = np.concatenate([[0, n_beams - 1], rng.integers(0, n_beams, size=n_decode_rows)])
        pick_h = np.concatenate([[0, w.n_q_heads - 1], rng.integers(0, w.n_q_heads, size=n_decode_rows)])
        rows = set(zip(pick_j.tolist(), pick_h.tolist()))
        jj, hh = np.array([r[0] for r in rows]), np.array([r[1] for r in rows])
        for layer in range(w.n_layers):
            dq, dk, dv = wl.decode_qkv(w, layer, step, "cuda")
            od = ses.decode_layer(layer, step, dq, dk, dv)
            ref = states[layer].step(to_np(dq), to_np(dk), to_np(dv), None, rows=rows)
            check(od.double().cpu().numpy()[jj, hh], ref[jj, hh], w.dtype,
                  f"{w.name} k={w.split_k} decode step {step} layer {layer}")
    assert ses.device_status() == 0
    # Eq. 9 on the buffers the session really holds
    earn, van = orc.kv_entries(lens, w.n_layers, w.split_k, R, generated=decode_steps)
    assert ses.kv_entries(decode_steps) == earn and van == w.n_layers * (int(lens.sum()) + w.batch * decode_steps)


@pytest.mark.parametrize("k", [0, 1, 2, 3, 4])
def test_split_layer_sweep_on_long_history_shapes(k):
    """The split sweep of the long-history workload changes which layers take which kernel: four layers of one
    4096-token prompt at every split from k = 0 (registers only from the first layer) to k = N (vanilla model)."""
    run_layer_mix(wl.CONFIGS["long"].replace(batch=1, n_layers=4, split_k=k))


def test_fullsize_1p5b():
    run_fullsize(wl.CONFIGS["1p5b"])


def test_fullsize_7b():
    run_fullsize(wl.CONFIGS["7b"])


def test_fullsize_long_history():
    # the split sweep k in {2, 4, 8, 16} changes how many layers take each kernel, not the kernels' shapes
    run_fullsize(wl.CONFIGS["long"], n_random=600, n_decode_rows=200)


def test_fullsize_ragged_beams():
    run_fullsize(wl.CONFIGS["ragged"], decode_steps=3, n_random=800, n_decode_rows=300)


def test_long_context_20k_tokens():
    # the paper pads prompts up to 20K tokens for its length study (Section 4, sequence-length scaling): 160 key
    # tiles per query tile in prefill, split-KV decode over a 20K-token prompt cache
    run_fullsize(wl.CONFIGS["long"].replace(name="20k", batch=2, prompt_len=20480, seed=6), n_random=500, n_decode_rows=150)


@pytest.mark.parametrize("name", ["paper_mha", "paper_gqa"])
def test_paper_operating_points(name):
    """The shapes the paper itself measures on: 50-200 token prompts, one register per side, beam 20, 4-token item
    identifiers; multi-head attention (two query tiles of a head per work item, 20 query rows per kv head) and a
    group of 7 (140 query rows per kv head: nine row tiles in three CTAs).  Every element is compared."""
    from parity_util import run_workload_and_compare
    run_workload_and_compare(wl.CONFIGS[name].replace(n_layers=2, split_k=1), check_lse=False)
