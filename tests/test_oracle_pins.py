"""Pins for the CPU oracle: each check compares it with something other than itself —
scalar brute force, a library routine, closed forms, invariants and the paper's worked example."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import earn_oracle as orc
from paper_2507_00715_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- helpers (independent of the oracle)
def brute_attention_row(q, keys, vals, scale):
    """Scalar loops, python floats, math.fsum: softmax(q.K^T * scale) V for one row."""
    logits = [math.fsum(q[d] * kk[d] for d in range(len(q))) * scale for kk in keys]
    m = max(logits)
    w = [math.exp(s - m) for s in logits]
    z = math.fsum(w)
    return [math.fsum(w[j] * vals[j][d] for j in range(len(keys))) / z for d in range(len(q))]


def brute_causal(q, k, v, cu, scale):
    total, hq, d = q.shape
    g = hq // k.shape[1]
    out = np.zeros((total, hq, d))
    for b in range(len(cu) - 1):
        for i in range(cu[b], cu[b + 1]):
            for h in range(hq):
                keys = [list(k[j, h // g]) for j in range(cu[b], i + 1)]
                vals = [list(v[j, h // g]) for j in range(cu[b], i + 1)]
                out[i, h] = brute_attention_row(list(q[i, h]), keys, vals, scale)
    return out


def rand_qkv(rng, total, hq, hkv, d):
    return (rng.standard_normal((total, hq, d)), rng.standard_normal((total, hkv, d)),
            rng.standard_normal((total, hkv, d)))


# ---------------------------------------------------------------- causal attention (Eq. 3 + mask)
def test_causal_matches_scalar_brute_force():
    rng = np.random.default_rng(0)
    cu = np.array([0, 5, 6, 14])
    q, k, v = rand_qkv(rng, 14, 4, 2, 3)
    o, lse = orc.causal_attention(q, k, v, cu)
    ref = brute_causal(q, k, v, cu, 1 / math.sqrt(3))
    np.testing.assert_allclose(o, ref, rtol=0, atol=1e-13)
    # LSE: recompute one entry by hand
    i, h = 9, 3
    logits = [float(q[i, h] @ k[j, 1]) / math.sqrt(3) for j in range(6, i + 1)]
    assert abs(lse[h, i] - math.log(math.fsum(math.exp(s) for s in logits))) < 1e-12


def test_causal_matches_library_sdpa():
    """With k = N every layer is ordinary causal attention: compare with torch's fp64 SDPA."""
    rng = np.random.default_rng(1)
    L, hq, hkv, d = 37, 6, 2, 16
    q, k, v = rand_qkv(rng, L, hq, hkv, d)
    o, _ = orc.causal_attention(q, k, v, [0, L])
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(k).permute(1, 0, 2)[None].repeat_interleave(hq // hkv, dim=1)
    tv = torch.from_numpy(v).permute(1, 0, 2)[None].repeat_interleave(hq // hkv, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0].permute(1, 0, 2).numpy()
    np.testing.assert_allclose(o, ref, rtol=0, atol=1e-12)


def test_closed_forms():
    rng = np.random.default_rng(2)
    L, hq, hkv, d = 9, 2, 1, 4
    q, k, v = rand_qkv(rng, L, hq, hkv, d)
    # zero queries -> uniform softmax -> running mean of V
    o, lse = orc.causal_attention(np.zeros_like(q), k, v, [0, L])
    run_mean = np.cumsum(v[:, 0, :], axis=0) / np.arange(1, L + 1)[:, None]
    np.testing.assert_allclose(o[:, 0], run_mean, atol=1e-14)
    np.testing.assert_allclose(lse[0], np.log(np.arange(1, L + 1)), atol=1e-14)
    # first row has one key -> O = V[0] whatever Q is
    o, _ = orc.causal_attention(q, k, v, [0, L])
    np.testing.assert_allclose(o[0, 1], v[0, 0], atol=1e-15)
    # a key that dominates by a huge margin selects its value row: plants catch a transposed operand
    k2 = k.copy()
    k2[3, 0] = 1000.0 * q[7, 0] / np.linalg.norm(q[7, 0])
    o, _ = orc.causal_attention(q, k2, v, [0, L])
    np.testing.assert_allclose(o[7, 0], v[3, 0], atol=1e-9)
    # scale: sqrt(head_dim).  With K = c*Q/|Q| logits are c*|Q|/sqrt(d); check through LSE of a 1-key row
    o1, lse1 = orc.causal_attention(q[:1], k[:1], v[:1], [0, 1])
    assert abs(lse1[0, 0] - float(q[0, 0] @ k[0, 0]) / math.sqrt(d)) < 1e-13
    # explicit scale overrides
    _, lse2 = orc.causal_attention(q[:1], k[:1], v[:1], [0, 1], scale=0.5)
    assert abs(lse2[1, 0] - float(q[0, 1] @ k[0, 0]) * 0.5) < 1e-13


def test_gqa_head_mapping_and_ragged_independence():
    rng = np.random.default_rng(3)
    lens = [4, 1, 7]
    cu = np.concatenate([[0], np.cumsum(lens)])
    q, k, v = rand_qkv(rng, cu[-1], 6, 3, 5)
    o, _ = orc.causal_attention(q, k, v, cu)
    # each sequence alone, each kv head expanded by hand
    for b in range(3):
        sl = slice(cu[b], cu[b + 1])
        for h in range(6):
            oo, _ = orc.causal_attention(q[sl, h:h + 1], k[sl, h // 2:h // 2 + 1], v[sl, h // 2:h // 2 + 1], [0, lens[b]])
            np.testing.assert_array_equal(oo[:, 0], o[sl, h])
    # batch permutation
    perm = [2, 0, 1]
    idx = np.concatenate([np.arange(cu[b], cu[b + 1]) for b in perm])
    cu_p = np.concatenate([[0], np.cumsum([lens[b] for b in perm])])
    op, _ = orc.causal_attention(q[idx], k[idx], v[idx], cu_p)
    np.testing.assert_array_equal(op, o[idx])


def test_rows_variant_matches_full():
    rng = np.random.default_rng(4)
    cu = np.array([0, 11, 30])
    q, k, v = rand_qkv(rng, 30, 4, 2, 8)
    o, _ = orc.causal_attention(q, k, v, cu)
    tok = [0, 10, 11, 29, 17]
    head = [0, 3, 2, 1, 0]
    rows = orc.causal_attention_rows(q, k, v, cu, tok, head)
    ref = brute_causal(q, k, v, cu, 1 / math.sqrt(8))
    for n, (t, h) in enumerate(zip(tok, head)):
        np.testing.assert_allclose(rows[n], ref[t, h], atol=1e-13)
        np.testing.assert_allclose(rows[n], o[t, h], atol=1e-13)


# ---------------------------------------------------------------- register indices / compaction
def test_register_indices_enumeration():
    for L in range(1, 9):
        for rh, rt in itertools.product(range(0, 5), range(0, 5)):
            if rh + rt > L:
                with pytest.raises(ValueError):
                    orc.register_indices([L], rh, rt)
                continue
            idx = orc.register_indices([L], rh, rt)[0]
            expect = list(range(L))[:rh] + (list(range(L))[L - rt:] if rt else [])
            assert list(idx) == expect
            assert all(idx[i] < idx[i + 1] for i in range(len(idx) - 1))
    # R == L: identity
    assert list(orc.register_indices([6], 2, 4)[0]) == list(range(6))


def test_compact_is_bit_copy():
    rng = np.random.default_rng(5)
    lens = [5, 9, 4]
    cu = np.concatenate([[0], np.cumsum(lens)])
    x = rng.standard_normal((cu[-1], 2, 3)).astype(np.float32)
    idx = orc.register_indices(lens, 1, 2)
    c = orc.compact(x, cu, idx)
    assert c.dtype == x.dtype and c.shape == (3, 3, 2, 3)
    for b in range(3):
        seq = x[cu[b]:cu[b + 1]]
        expect = np.stack([seq[0], seq[-2], seq[-1]])
        assert c[b].tobytes() == expect.tobytes()


# ---------------------------------------------------------------- register layers
@pytest.mark.parametrize("rh,rt", [(2, 2), (0, 3), (3, 0), (1, 1), (4, 1)])
def test_form_a_equals_form_b(rh, rt):
    rng = np.random.default_rng(6)
    lens = [12, rh + rt, rh + rt + 1]
    cu = np.concatenate([[0], np.cumsum(lens)])
    q, k, v = rand_qkv(rng, cu[-1], 4, 2, 6)
    idx = orc.register_indices(lens, rh, rt)
    a = orc.register_attention(orc.compact(q, cu, idx), orc.compact(k, cu, idx), orc.compact(v, cu, idx))
    b = orc.register_attention_masked(q, k, v, cu, idx)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-13)


def test_form_b_matches_scalar_brute_force():
    rng = np.random.default_rng(7)
    L, rh, rt = 8, 2, 1
    q, k, v = rand_qkv(rng, L, 2, 1, 2)
    idx = orc.register_indices([L], rh, rt)
    got = orc.register_attention_masked(q, k, v, [0, L], idx)
    regs = [0, 1, 7]
    for m, i in enumerate(regs):
        js = [j for j in regs if j <= i]
        for h in range(2):
            ref = brute_attention_row(list(q[i, h]), [list(k[j, 0]) for j in js], [list(v[j, 0]) for j in js],
                                      1 / math.sqrt(2))
            np.testing.assert_allclose(got[0, m, h], ref, atol=1e-13)


def test_register_layers_ignore_prompt_tokens():
    """Layers after the split depend on register K/V only: overwrite every other row with noise and
    the compact cache, the register outputs and all decode outputs stay bit-identical."""
    w = wl.CONFIGS["tiny"].replace(prompt_len=40, decode_steps=3)
    cu = wl.cu_seqlens(w)
    q, k, v = (t.numpy() for t in wl.layer_qkv(w, 3))
    idx = orc.register_indices(wl.seqlens(w), w.r_head, w.r_tail)

    def run(q, k, v):
        kc, vc, qc = orc.compact(k, cu, idx), orc.compact(v, cu, idx), orc.compact(q, cu, idx)
        o = orc.register_attention(qc, kc, vc)
        st = orc.DecodeState([kc[0]], [vc[0]], 1)
        outs = []
        for s in range(1, 4):
            dq, dk, dv = (t.numpy() for t in wl.decode_qkv(w, 3, s))
            outs.append(st.step(dq, dk, dv))
        return kc, vc, o, np.stack(outs)

    base = run(q, k, v)
    rng = np.random.default_rng(8)
    keep = np.zeros(40, dtype=bool)
    keep[idx[0]] = True
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    for t in (q2, k2, v2):
        t[~keep] = rng.standard_normal(t[~keep].shape).astype(t.dtype)
    pert = run(q2, k2, v2)
    for a, b in zip(base, pert):
        assert a.tobytes() == b.tobytes()
    # and the masked form agrees on the perturbed input too
    np.testing.assert_allclose(orc.register_attention_masked(q2, k2, v2, cu, idx), base[2], atol=1e-13)


# ---------------------------------------------------------------- decode (Eq. 4)
def test_decode_step_is_last_row_of_causal_prefill():
    rng = np.random.default_rng(9)
    L, hq, hkv, d, T = 10, 4, 2, 4, 3
    q, k, v = rand_qkv(rng, L, hq, hkv, d)
    dq, dk, dv = rand_qkv(rng, T, hq, hkv, d)
    st = orc.DecodeState([k], [v], 1)
    for s in range(1, T + 1):
        o = st.step(dq[s - 1:s], dk[s - 1:s], dv[s - 1:s])
        qq = np.concatenate([q, dq[:s]])
        kk = np.concatenate([k, dk[:s]])
        vv = np.concatenate([v, dv[:s]])
        ref, _ = orc.causal_attention(qq, kk, vv, [0, L + s])
        np.testing.assert_allclose(o[0], ref[-1], atol=1e-13)
        assert st.entries(0) == L + s                       # cache length after append
    # brute-force the last step as well
    ref = brute_attention_row(list(dq[T - 1, 3]), [list(x) for x in np.concatenate([k, dk])[:, 1]],
                              [list(x) for x in np.concatenate([v, dv])[:, 1]], 0.5)
    np.testing.assert_allclose(o[0, 3], ref, atol=1e-13)


def test_beams_equal_independent_runs():
    rng = np.random.default_rng(10)
    B, W, R, hq, hkv, d, T = 2, 3, 4, 2, 1, 4, 4
    kc = [rng.standard_normal((R, hkv, d)) for _ in range(B)]
    vc = [rng.standard_normal((R, hkv, d)) for _ in range(B)]
    dq = rng.standard_normal((T, B * W, hq, d))
    dk = rng.standard_normal((T, B * W, hkv, d))
    dv = rng.standard_normal((T, B * W, hkv, d))
    parents = [None] + [rng.integers(0, W, size=B * W) for _ in range(T - 1)]
    st = orc.DecodeState(kc, vc, W)
    outs = [st.step(dq[s], dk[s], dv[s], parents[s]) for s in range(T)]
    # follow each final beam's lineage by hand and run it as a single-beam problem
    for j in range(B * W):
        b = j // W
        chain = [j]
        for s in range(T - 1, 0, -1):
            chain.append(b * W + int(parents[s][chain[-1]]))
        chain = chain[::-1]                                   # chain[s] = physical beam that produced token s
        solo = orc.DecodeState([kc[b]], [vc[b]], 1)
        for s in range(T):
            c = chain[s]
            o = solo.step(dq[s, j if s == T - 1 else c][None], dk[s, c][None], dv[s, c][None])
        np.testing.assert_allclose(o[0], outs[T - 1][j], atol=1e-13)


# ---------------------------------------------------------------- accounting (Eq. 8, 9, 13)
def _golden():
    vals = {}
    with open(os.path.join(GOLDEN, "worked_example.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if len(line) == 2:
                vals[line[0]] = float(line[1])
    return vals


def test_worked_example_of_the_paper():
    g = _golden()
    N, L, k, r = int(g["N"]), int(g["L"]), int(g["k"]), int(g["r"])
    gc = orc.gamma_cache(N, k, L, r)
    assert abs(100 * gc - g["gamma_cache_percent"]) <= 0.5
    sp = orc.speedup(N, k, L, r, int(g["n_h"]), int(g["d_a"]), int(g["d_h"]), int(g["d_f"]))
    assert abs(sp - g["speedup"]) <= 0.1
    # the two printed forms of Eq. 9 agree, and the count form N_KV = n_h (kL + (N-k) r) gives the same ratio
    assert abs(gc - (N - k) * (L - r) / (N * L)) < 1e-15
    earn, van = orc.kv_entries([L] * 3, N, k, r, n_kv_heads=int(g["n_h"]))
    assert earn == 3 * int(g["n_h"]) * (k * L + (N - k) * r) and van == 3 * int(g["n_h"]) * N * L
    assert abs((1 - earn / van) - gc) < 1e-15
    # Eq. 8 is about k/N and Eq. 13 about N/k
    ga = orc.gamma_attn(N, k, L, r, 32, 128, 4096, 11008)
    assert abs(ga - k / N) < 0.01 and abs(sp - N / k) < 0.1
    # Eq. 18 against its expanded form, Eq. 16 + Eq. 17
    assert orc.layer_flops(L, 32, 128, 4096, 11008) == 32 * (8 * L * 4096 * 128 + 4 * L * L * 128) + 4 * L * 4096 * 11008


def test_compact_cache_size_is_registers_plus_generated():
    w = wl.CONFIGS["tiny"]
    cu = wl.cu_seqlens(w)
    _, k, v = (t.numpy() for t in wl.layer_qkv(w, 2))
    idx = orc.register_indices(wl.seqlens(w), w.r_head, w.r_tail)
    kc, vc = orc.compact(k, cu, idx), orc.compact(v, cu, idx)
    late = orc.DecodeState([kc[0]], [vc[0]], 1)
    early = orc.DecodeState([k], [v], 1)
    for s in range(1, 4):
        dq, dk, dv = (t.numpy() for t in wl.decode_qkv(w, 2, s))
        late.step(dq, dk, dv)
        early.step(dq, dk, dv)
        assert late.entries(0) == w.n_regs + s
        assert early.entries(0) == w.prompt_len + s
    earn, van = orc.kv_entries(wl.seqlens(w), w.n_layers, w.split_k, w.n_regs)
    assert abs((1 - earn / van) - orc.gamma_cache(w.n_layers, w.split_k, w.prompt_len, w.n_regs)) < 1e-15
    assert abs(100 * (1 - earn / van) - 48.4375) < 1e-9       # (N-k)(L-r)/(NL) = 2*248/(4*256)


# ---------------------------------------------------------------- diagnostics (Eq. 14-15) and the input recipe
def test_diagnostics_definitions():
    p = np.array([0.5, 0.04, 0.06, 0.1, 0.05, 0.05, 0.2])
    assert orc.sparsity(p) == pytest.approx(4 / 7)            # strictly above 0.05
    head, tail = orc.sinks(p)
    assert head == pytest.approx(0.6) and tail == pytest.approx(0.4)   # first 3; positions n-3..n


def test_synthetic_inputs_show_dual_sinks():
    w = wl.CONFIGS["tiny"]
    q, k, _ = (t.numpy() for t in wl.layer_qkv(w, 0))
    heads, tails = [], []
    for h in range(w.n_q_heads):
        p = orc.attention_scores(q[-1, h], k[:, h // w.group])
        a, b = orc.sinks(p)
        heads.append(a)
        tails.append(b)
    # 2 sink keys of weight ~e^4 among 256 ordinary ones: each side holds a visible share
    assert np.mean(heads) > 0.08 and np.mean(tails) > 0.08


# ---- the hidden-state form of the register-focused process (gather X -> X', then Eq. 2 on the register rows)
def test_rms_norm_and_rope_closed_forms():
    x = np.full((3, 8), 2.0)
    assert np.allclose(orc.rms_norm(x, np.arange(8.0), 0.0), np.tile(np.arange(8.0), (3, 1)))     # x / |x|_rms = 1
    cos, sin = orc.rope_tables(16, 8)
    v = np.random.default_rng(0).standard_normal((5, 8))
    assert np.allclose(orc.apply_rope(v, cos[0], sin[0]), v)                                       # position 0: identity
    for pos in (1, 7, 15):
        assert np.allclose(np.linalg.norm(orc.apply_rope(v, cos[pos], sin[pos]), axis=-1), np.linalg.norm(v, axis=-1))
    # the score of a rotated query and key depends on the distance between their positions only
    q, k = v[0], v[1]
    s1 = orc.apply_rope(q, cos[9], sin[9]) @ orc.apply_rope(k, cos[4], sin[4])
    s2 = orc.apply_rope(q, cos[14], sin[14]) @ orc.apply_rope(k, cos[9], sin[9])
    assert np.isclose(s1, s2)
    # lowest pair at position p is a plane rotation by p radians (theta^0 = 1)
    r = orc.apply_rope(np.array([1.0, 0, 0, 0, 0.0, 0, 0, 0]), cos[3], sin[3])
    assert np.allclose([r[0], r[4]], [np.cos(3.0), np.sin(3.0)])


def test_register_qkv_matches_library_ops_and_commutes_with_the_gather():
    rng = np.random.default_rng(5)
    lens, rh, rt, dm, hq, hkv, d = (9, 6), 2, 1, 32, 4, 2, 8
    cu = np.concatenate([[0], np.cumsum(lens)])
    x = rng.standard_normal((cu[-1], dm))
    wn = rng.standard_normal(dm)
    w = rng.standard_normal(((hq + 2 * hkv) * d, dm)) / np.sqrt(dm)
    cos, sin = orc.rope_tables(16, d)
    idx = orc.register_indices(lens, rh, rt)
    q, k, v = orc.register_qkv(x, cu, idx, wn, w, hq, hkv, d, cos, sin, eps=1e-6)
    # library: normalise and project EVERY token, rotate by its own position, then gather the register rows
    xt = torch.from_numpy(x)
    y = torch.nn.functional.linear(torch.nn.functional.rms_norm(xt, (dm,), torch.from_numpy(wn), 1e-6), torch.from_numpy(w)).numpy()
    for b in range(2):
        for m in range(rh + rt):
            pos = idx[b, m]
            row = y[cu[b] + pos]
            assert np.allclose(q[b, m], orc.apply_rope(row[:hq * d].reshape(hq, d), cos[pos], sin[pos]))
            assert np.allclose(k[b, m], orc.apply_rope(row[hq * d:(hq + hkv) * d].reshape(hkv, d), cos[pos], sin[pos]))
            assert np.allclose(v[b, m], row[(hq + hkv) * d:].reshape(hkv, d))
    # rows outside the registers do not matter
    x2 = x.copy()
    keep = np.zeros(cu[-1], bool)
    for b in range(2):
        keep[cu[b] + idx[b]] = True
    x2[~keep] = rng.standard_normal((int((~keep).sum()), dm))
    q2, k2, v2 = orc.register_qkv(x2, cu, idx, wn, w, hq, hkv, d, cos, sin, eps=1e-6)
    assert np.array_equal(q, q2) and np.array_equal(k, k2) and np.array_equal(v, v2)


# ---------------------------------------------------------------- sampled-row decode, rotary frequencies, scores
def test_decode_step_with_sampled_rows_equals_the_plain_step():
    """The sampled-row form of DecodeState.step (used where a workload is too large to compute in full) must keep
    the cache exactly as the plain step does -- every beam appended and re-parented, selected or not -- and return
    the plain step's values on the selected rows, zeros elsewhere (Eq. 4; Section 3.2 decoding rule)."""
    rng = np.random.default_rng(11)
    B, W, R, hq, hkv, d, T = 2, 3, 5, 4, 2, 4, 4
    kc = [rng.standard_normal((R, hkv, d)) for _ in range(B)]
    vc = [rng.standard_normal((R, hkv, d)) for _ in range(B)]
    full, part = orc.DecodeState(kc, vc, W), orc.DecodeState(kc, vc, W)
    for s in range(T):
        dq = rng.standard_normal((B * W, hq, d))
        dk = rng.standard_normal((B * W, hkv, d))
        dv = rng.standard_normal((B * W, hkv, d))
        parents = None if s == 0 else rng.integers(0, W, size=B * W)
        # a different selection every step, so that a beam skipped at one step is read (through a child) at a later one
        rows = {(int(j), int(h)) for j, h in zip(rng.integers(0, B * W, size=4), rng.integers(0, hq, size=4))}
        o_full = full.step(dq, dk, dv, parents)
        o_part = part.step(dq, dk, dv, parents, rows=rows)
        for j in range(B * W):
            for h in range(hq):
                if (j, h) in rows:
                    assert np.array_equal(o_part[j, h], o_full[j, h])
                else:
                    assert not o_part[j, h].any()
        for j in range(B * W):
            assert len(part.priv_k[j]) == len(full.priv_k[j]) == s + 1
            assert np.array_equal(np.stack(part.priv_k[j]), np.stack(full.priv_k[j]))
            assert np.array_equal(np.stack(part.priv_v[j]), np.stack(full.priv_v[j]))
        assert [part.entries(b) for b in range(B)] == [full.entries(b) for b in range(B)] == [R + s + 1] * B
    # and the selected rows are right by themselves: one of them against the scalar brute force
    j, h = next(iter(rows))
    keys = np.concatenate([kc[j // W][:, h // 2], np.stack(full.priv_k[j])[:, h // 2]])
    vals = np.concatenate([vc[j // W][:, h // 2], np.stack(full.priv_v[j])[:, h // 2]])
    ref = brute_attention_row(list(dq[j, h]), [list(x) for x in keys], [list(x) for x in vals], 0.5)
    np.testing.assert_allclose(o_part[j, h], ref, atol=1e-13)


def test_rope_frequency_ladder_closed_form():
    """Pair i turns by pos * theta^(-2i/D): with D = 8 and theta = 10000 the four pairs turn by 1, 0.1, 0.01 and
    0.001 radians per position (any other exponent on the ladder fails here)."""
    cos, sin = orc.rope_tables(8, 8, theta=10000.0)
    for pos in (1, 5):
        np.testing.assert_allclose(cos[pos], np.cos(pos * np.array([1.0, 0.1, 0.01, 0.001])), atol=1e-15)
        np.testing.assert_allclose(sin[pos], np.sin(pos * np.array([1.0, 0.1, 0.01, 0.001])), atol=1e-15)
    # D = 4, theta = 16: pairs turn by 1 and 16^(-1/2) = 0.25 radians per position
    cos, sin = orc.rope_tables(3, 4, theta=16.0)
    np.testing.assert_allclose(sin[2], [math.sin(2.0), math.sin(0.5)], atol=1e-15)
    # the pair (i, i + D/2) is what turns: unit vector on coordinate 1 of D = 8 moves into coordinate 5
    r = orc.apply_rope(np.array([0.0, 1, 0, 0, 0, 0, 0, 0]), *(t[1] for t in orc.rope_tables(2, 8)))
    np.testing.assert_allclose([r[1], r[5]], [math.cos(0.1), math.sin(0.1)], atol=1e-15)
    assert not r[[0, 2, 3, 4, 6, 7]].any()


def test_attention_scores_by_hand():
    """Eq. 14-15 take the softmax scores of one row: compare with the scalar definition."""
    rng = np.random.default_rng(12)
    qrow, keys = rng.standard_normal(6), rng.standard_normal((7, 6))
    p = orc.attention_scores(qrow, keys)
    logits = [math.fsum(qrow[d] * keys[j][d] for d in range(6)) / math.sqrt(6) for j in range(7)]
    z = math.fsum(math.exp(s) for s in logits)
    np.testing.assert_allclose(p, [math.exp(s) / z for s in logits], atol=1e-15)
    assert abs(p.sum() - 1.0) < 1e-15


# ---------------------------------------------------------------- beam selection (Appendix A.3: beam search)
def test_beam_topk_matches_sorted_tuples_and_hand_cases():
    rng = np.random.default_rng(13)
    B, W, V = 3, 4, 11
    lp = rng.standard_normal((B * W, V)).astype(np.float32)
    lp[2, 5] = lp[1, 3] = lp[0, 7]                      # plant exact ties inside sequence 0 (equal beam scores below)
    sc = rng.standard_normal(B * W).astype(np.float32)
    sc[0] = sc[1] = sc[2]
    parent, token, score = orc.beam_topk(lp, sc, W)
    for b in range(B):
        cands = []
        for w in range(W):
            for v in range(V):
                cands.append((-float(np.float32(sc[b * W + w]) + np.float32(lp[b * W + w, v])), w * V + v))
        best = sorted(cands)[:W]                        # higher score first, then lower flat index
        assert [c[1] // V for c in best] == list(parent[b * W:(b + 1) * W])
        assert [c[1] % V for c in best] == list(token[b * W:(b + 1) * W])
        assert [np.float32(-c[0]) for c in best] == list(score[b * W:(b + 1) * W])
    # one beam far ahead of the others: every survivor continues it, tokens in order of their log-probability
    sc2 = np.array([0.0, 100.0, 0.0, 0.0], dtype=np.float32)
    lp2 = rng.standard_normal((4, 9)).astype(np.float32)
    p2, t2, s2 = orc.beam_topk(lp2, sc2, 4)
    assert list(p2) == [1, 1, 1, 1] and list(t2) == list(np.argsort(-lp2[1], kind="stable")[:4])
    # all candidates equal: the first W flat indices, in order
    p3, t3, s3 = orc.beam_topk(np.zeros((3, 5), np.float32), np.zeros(3, np.float32), 3)
    assert list(p3) == [0, 0, 0] and list(t3) == [0, 1, 2] and not s3.any()
    # first step: only beam 0 is live, whatever the other rows hold
    lp4 = rng.standard_normal((4, 9)).astype(np.float32)
    lp4[1:] += 50.0
    p4, t4, _ = orc.beam_topk(lp4, np.zeros(4, np.float32), 4, n_live=1)
    assert list(p4) == [0, 0, 0, 0] and list(t4) == list(np.argsort(-lp4[0], kind="stable")[:4])
    # one beam: greedy decoding, the arg max
    lp5 = rng.standard_normal((6, 13)).astype(np.float32)
    p5, t5, s5 = orc.beam_topk(lp5, np.zeros(6, np.float32), 1)
    assert not p5.any() and list(t5) == list(lp5.argmax(axis=1)) and np.array_equal(s5, lp5.max(axis=1))
    with pytest.raises(ValueError):
        orc.beam_topk(np.zeros((4, 3), np.float32), np.zeros(4, np.float32), 4, n_live=1)   # 3 candidates for 4 slots


# ---------------------------------------------------------------- training (Section 3.2 "Training", Eq. 7)
def _torch_masked_attention(q, k, v, allowed):
    """Dense attention of one sequence in torch fp64 under an explicit boolean mask [n, n] (library softmax / matmul),
    GQA heads expanded by hand: q [n,Hq,D], k, v [n,Hkv,D] tensors that require grad."""
    hq, hkv, d = q.shape[1], k.shape[1], q.shape[2]
    kk = k.repeat_interleave(hq // hkv, dim=1)
    vv = v.repeat_interleave(hq // hkv, dim=1)
    s = torch.einsum("ihd,jhd->hij", q, kk) / math.sqrt(d)
    s = s.masked_fill(~allowed[None], float("-inf"))
    return torch.einsum("hij,jhd->ihd", torch.softmax(s, dim=-1), vv)


def test_causal_attention_grad_matches_finite_differences_and_autograd():
    rng = np.random.default_rng(14)
    cu = np.array([0, 5, 6, 13])
    q, k, v = rand_qkv(rng, 13, 4, 2, 3)
    go = rng.standard_normal(q.shape)
    dq, dk, dv = orc.causal_attention_grad(q, k, v, cu, go)
    loss = lambda q_, k_, v_: float(np.sum(orc.causal_attention(q_, k_, v_, cu)[0] * go))   # noqa: E731
    eps = 1e-6
    for arr, grad, which in ((q, dq, 0), (k, dk, 1), (v, dv, 2)):
        for _ in range(12):                                    # sampled coordinates, central differences
            i = tuple(int(rng.integers(0, n)) for n in arr.shape)
            hi, lo = arr.copy(), arr.copy()
            hi[i] += eps
            lo[i] -= eps
            args_hi = [q, k, v]
            args_lo = [q, k, v]
            args_hi[which], args_lo[which] = hi, lo
            fd = (loss(*args_hi) - loss(*args_lo)) / (2 * eps)
            assert abs(fd - grad[i]) < 1e-7, (which, i, fd, grad[i])
    # k = N: every layer is ordinary causal attention; torch autograd through the library SDPA, sequence by sequence
    for b in range(3):
        sl = slice(cu[b], cu[b + 1])
        tq, tk, tv = (torch.from_numpy(x[sl]).clone().requires_grad_(True) for x in (q, k, v))
        o = torch.nn.functional.scaled_dot_product_attention(
            tq.permute(1, 0, 2)[None], tk.permute(1, 0, 2)[None].repeat_interleave(2, dim=1),
            tv.permute(1, 0, 2)[None].repeat_interleave(2, dim=1), is_causal=True)[0].permute(1, 0, 2)
        (o * torch.from_numpy(go[sl])).sum().backward()
        np.testing.assert_allclose(dq[sl], tq.grad.numpy(), atol=1e-12)
        np.testing.assert_allclose(dk[sl], tk.grad.numpy(), atol=1e-12)
        np.testing.assert_allclose(dv[sl], tv.grad.numpy(), atol=1e-12)


@pytest.mark.parametrize("rh,rt,nt", [(2, 1, 3), (0, 2, 4), (1, 0, 1), (2, 2, 0)])
def test_training_rule_for_layers_after_the_split(rh, rt, nt):
    """Layers l > k of a training sample: only register and target tokens take part.  Stated as a mask on a dense
    full-length attention (keys restricted to the participating set, causal) and differentiated by torch autograd, it
    gives on the participating rows what the oracle computes on the gathered rows, the same gradients there, and no
    gradient at all on the prompt rows."""
    rng = np.random.default_rng(15)
    lens = [11, rh + rt + nt + 1, rh + rt + nt]
    cu = np.concatenate([[0], np.cumsum(lens)])
    q, k, v = rand_qkv(rng, cu[-1], 4, 2, 5)
    idx = orc.participating_indices(lens, rh, rt, nt)
    P = rh + rt + nt
    for b, L in enumerate(lens):                              # the layout [prefix; ...; suffix; targets] by hand
        assert list(idx[b]) == list(range(rh)) + list(range(L - nt - rt, L))
    q_p, k_p, v_p = orc.compact(q, cu, idx), orc.compact(k, cu, idx), orc.compact(v, cu, idx)
    go_p = rng.standard_normal(q_p.shape)
    o_p, lse_p = orc.participating_attention(q_p, k_p, v_p)
    dq_p, dk_p, dv_p = orc.participating_attention_grad(q_p, k_p, v_p, go_p)
    assert o_p.shape == (3, P, 4, 5) and lse_p.shape == (3, 4, P)
    for b, L in enumerate(lens):
        sl = slice(cu[b], cu[b + 1])
        tq, tk, tv = (torch.from_numpy(x[sl]).clone().requires_grad_(True) for x in (q, k, v))
        part = torch.zeros(L, dtype=torch.bool)
        part[torch.from_numpy(idx[b]).long()] = True
        allowed = torch.tril(torch.ones(L, L, dtype=torch.bool)) & part[None, :]
        allowed |= torch.eye(L, dtype=torch.bool) & ~part[:, None]       # prompt rows (unused) keep one key: no empty row
        o = _torch_masked_attention(tq, tk, tv, allowed)
        rows = torch.from_numpy(idx[b]).long()
        np.testing.assert_allclose(o[rows].detach().numpy(), o_p[b], atol=1e-12)
        (o[rows] * torch.from_numpy(go_p[b])).sum().backward()           # the loss sees the participating rows only
        for grad_p, t in ((dq_p, tq), (dk_p, tk), (dv_p, tv)):
            full = t.grad.numpy()
            np.testing.assert_allclose(full[idx[b]], grad_p[b], atol=1e-12)
            rest = np.ones(L, bool)
            rest[idx[b]] = False
            assert not full[rest].any()                                    # removed tokens receive no gradient
    # LSE of one row by hand
    b, m, h = 0, P - 1, 3
    logits = [float(q_p[b, m, h] @ k_p[b, j, 1]) / math.sqrt(5) for j in range(P)]
    assert abs(lse_p[b, h, m] - math.log(math.fsum(math.exp(x) for x in logits))) < 1e-12
