"""CPU fp64 oracle for the EARN attention path.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may call
this module; the product path (the CUDA library and its binding) never does,
and this module imports nothing from it.

Every function is the plain definition from the paper written out in numpy
float64, one (sequence, head) at a time, with no blocking, fusion or online
rescaling.  Inputs may be float32 or float64 arrays (bf16 tensors are widened
exactly by the caller); all arithmetic is float64.

What pins each function (see tests/test_oracle_pins.py):
  causal_attention      : brute-force scalar loops, a library SDPA call, closed
                          forms (zero queries -> running mean of V; one key -> V)
  register_indices      : enumeration on tiny lengths; Eq. 5 layout
  compact               : bit copies checked against python indexing
  register_attention    : form A (gathered, Section 3.2 inference) must equal
                          form B (masked full-length, Section 3.2 training rule)
  DecodeState / decode_attention : step s equals the last row of a causal prefill
                          over prompt ++ generated; W beams equal W independent runs;
                          the sampled-row form of step() leaves the same cache and the
                          same values on the selected rows as the plain form
  kv_entries, gamma_cache, gamma_attn, speedup : the worked example of Section 3.3
  rms_norm, apply_rope, register_qkv : closed forms (constant rows, zero angle, norm preservation), the
                          relative-position property of the rotation, a library rms_norm / linear call, and
                          "project every row then gather" = "gather then project" (Eq. 2 acts per token)
  rope_tables           : closed-form angles (D = 8, theta = 10000: 1, 0.1, 0.01, 0.001 rad per position)
  attention_scores, sparsity, sinks : the scalar definitions of Eq. 14-15 by hand
  causal_attention_grad : central finite differences of a scalar loss through causal_attention; torch autograd (fp64)
                          through a library SDPA call (with k = N training is ordinary causal attention)
  participating_attention(_grad), participating_indices : autograd through a dense full-length attention whose mask
                          is the training rule itself (keys restricted to the participating set) gives the same outputs
                          on the participating rows and the same gradients, zero on every prompt row
  beam_topk             : python's sorted() on (score, index) tuples; hand-made cases (a dominant beam, exact ties,
                          the first step with one live beam); greedy decoding (one beam) = argmax
Attention values have no printed worked example in the paper, so beyond those
pins they are parity unpinned.
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence, Tuple

import numpy as np


# --------------------------------------------------------------------------
# Eq. 5 (input layout X = [R_prefix; Prompt; R_suffix]) and the inference rule
# X -> X' = [X_prefix; X_suffix] of Section 3.2.
# --------------------------------------------------------------------------
def register_indices(seqlens: Sequence[int], r_head: int, r_tail: int) -> np.ndarray:
    """Positions (within each sequence) of the register tokens, int32 [B, r_head+r_tail].

    The prefix registers are the first r_head positions, the suffix registers
    the last r_tail positions; the order [prefix; suffix] is kept.
    """
    if r_head < 0 or r_tail < 0:
        raise ValueError("negative register count")
    out = np.zeros((len(seqlens), r_head + r_tail), dtype=np.int32)
    for b, L in enumerate(seqlens):
        L = int(L)
        if r_head + r_tail > L:
            raise ValueError(f"sequence {b}: {r_head}+{r_tail} registers exceed length {L}")
        for m in range(r_head):
            out[b, m] = m
        for m in range(r_tail):
            out[b, r_head + m] = L - r_tail + m
    return out


def _scale(d: int, scale: Optional[float]) -> float:
    # Eq. 3: logits are divided by sqrt(d), d the per-head dimension.
    return 1.0 / math.sqrt(d) if scale is None or scale == 0 else float(scale)


def _softmax_rows(s: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Row softmax of a float64 matrix with -inf for disallowed entries; returns (P, logsumexp)."""
    m = np.max(s, axis=1, keepdims=True)
    p = np.exp(s - m)
    z = np.sum(p, axis=1, keepdims=True)
    return p / z, (m + np.log(z))[:, 0]


# --------------------------------------------------------------------------
# Eq. 3 with the causal mask of a decoder-only model (layers l < k: all tokens).
# --------------------------------------------------------------------------
def causal_attention(q, k, v, cu_seqlens, scale: Optional[float] = None):
    """O[i] = sum_{j<=i} softmax_j(Q[i].K[j] * scale) V[j], per sequence and per query head.

    q [total,Hq,D]; k,v [total,Hkv,D]; query head h reads kv head h // (Hq/Hkv).
    Returns (O float64 [total,Hq,D], LSE float64 [Hq,total]) with LSE the natural
    log of the softmax denominator of the scaled logits.
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    total, hq, d = q.shape
    hkv = k.shape[1]
    g = hq // hkv
    sc = _scale(d, scale)
    o = np.zeros((total, hq, d), dtype=np.float64)
    lse = np.zeros((hq, total), dtype=np.float64)
    for b in range(len(cu_seqlens) - 1):
        lo, hi = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        n = hi - lo
        if n == 0:
            continue
        allowed = np.tril(np.ones((n, n), dtype=bool))          # j <= i
        for h in range(hq):
            s = (q[lo:hi, h, :] @ k[lo:hi, h // g, :].T) * sc
            s = np.where(allowed, s, -np.inf)
            p, l = _softmax_rows(s)
            o[lo:hi, h, :] = p @ v[lo:hi, h // g, :]
            lse[h, lo:hi] = l
    return o, lse


def causal_attention_rows(q, k, v, cu_seqlens, tok: Sequence[int], head: Sequence[int],
                          scale: Optional[float] = None) -> np.ndarray:
    """The same definition evaluated only for sampled (global token, query head) rows.

    Returns float64 [len(tok), D].  Used where the full result is too large to
    compute on the CPU; each row is computed on its own from Eq. 3.
    """
    cu = np.asarray(cu_seqlens)
    hq, d = q.shape[1], q.shape[2]
    g = hq // k.shape[1]
    sc = _scale(d, scale)
    out = np.zeros((len(tok), d), dtype=np.float64)
    for n, (t, h) in enumerate(zip(tok, head)):
        b = int(np.searchsorted(cu, t, side="right") - 1)
        lo = int(cu[b])
        qi = np.asarray(q[t, h, :], dtype=np.float64)
        kk = np.asarray(k[lo:t + 1, h // g, :], dtype=np.float64)
        vv = np.asarray(v[lo:t + 1, h // g, :], dtype=np.float64)
        s = (kk @ qi) * sc
        p = np.exp(s - np.max(s))
        out[n] = (p @ vv) / np.sum(p)
    return out


# --------------------------------------------------------------------------
# Section 3.2, inference, register-focused process: keep only register rows.
# --------------------------------------------------------------------------
def compact(x, cu_seqlens, idx: np.ndarray) -> np.ndarray:
    """Gather rows idx[b] of every sequence: x [total,H,D] -> [B,R,H,D], bit copies (dtype kept)."""
    x = np.asarray(x)
    b_, r_ = idx.shape
    out = np.zeros((b_, r_) + x.shape[1:], dtype=x.dtype)
    for b in range(b_):
        for m in range(r_):
            out[b, m] = x[int(cu_seqlens[b]) + int(idx[b, m])]
    return out


def register_attention(q_reg, k_reg, v_reg, scale: Optional[float] = None) -> np.ndarray:
    """Form A (Section 3.2, X' = [X_prefix; X_suffix]): causal attention among the R register
    tokens of each sequence in compact order.  q_reg [B,R,Hq,D], k_reg,v_reg [B,R,Hkv,D] -> [B,R,Hq,D].
    """
    b_, r_, hq, d = q_reg.shape
    if r_ == 0:
        return np.zeros((b_, 0, hq, d), dtype=np.float64)
    cu = np.arange(b_ + 1, dtype=np.int64) * r_
    o, _ = causal_attention(np.asarray(q_reg).reshape(b_ * r_, hq, d),
                            np.asarray(k_reg).reshape(b_ * r_, -1, d),
                            np.asarray(v_reg).reshape(b_ * r_, -1, d), cu, scale)
    return o.reshape(b_, r_, hq, d)


def register_attention_masked(q, k, v, cu_seqlens, idx: np.ndarray, scale: Optional[float] = None) -> np.ndarray:
    """Form B (Section 3.2, training rule for layers l > k): full-length attention in which only
    register tokens participate: allowed(i, j) = (j <= i) and j is a register position.
    Rows at register positions are returned, [B,R,Hq,D] float64.
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    hq, d = q.shape[1], q.shape[2]
    g = hq // k.shape[1]
    sc = _scale(d, scale)
    b_, r_ = idx.shape
    out = np.zeros((b_, r_, hq, d), dtype=np.float64)
    for b in range(b_):
        lo, hi = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        n = hi - lo
        is_reg = np.zeros(n, dtype=bool)
        is_reg[idx[b]] = True
        allowed = np.tril(np.ones((n, n), dtype=bool)) & is_reg[None, :]
        for h in range(hq):
            s = (q[lo:hi, h, :] @ k[lo:hi, h // g, :].T) * sc
            s = np.where(allowed, s, -np.inf)
            for m in range(r_):
                i = int(idx[b, m])
                row = s[i]
                p = np.exp(row - np.max(row))
                out[b, m, h] = (p @ v[lo:hi, h // g, :]) / np.sum(p)
    return out


# --------------------------------------------------------------------------
# Section 3.2, inference, register-focused process, as the paper states it: the HIDDEN STATE entering
# layer k is cut down to the register rows, X -> X' = [X_prefix; X_suffix], and only those rows go through
# the layer.  Eq. 2 (Q = X W_Q, K = X W_K, V = X W_V) applied to the gathered rows, inside a pre-norm
# decoder layer with rotary position embedding; the registers keep their original positions.
# --------------------------------------------------------------------------
def rms_norm(x: np.ndarray, weight: np.ndarray, eps: float) -> np.ndarray:
    """y = x / sqrt(mean(x^2) + eps) * weight over the last axis, float64."""
    x = np.asarray(x, dtype=np.float64)
    return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps) * np.asarray(weight, dtype=np.float64)


def rope_tables(max_pos: int, head_dim: int, theta: float = 10000.0) -> Tuple[np.ndarray, np.ndarray]:
    """cos / sin of pos * theta^(-2i/D), i < D/2: float64 [max_pos, D/2]."""
    inv = theta ** (-np.arange(0, head_dim, 2, dtype=np.float64) / head_dim)
    ang = np.arange(max_pos, dtype=np.float64)[:, None] * inv[None, :]
    return np.cos(ang), np.sin(ang)


def apply_rope(v: np.ndarray, cos: np.ndarray, sin: np.ndarray) -> np.ndarray:
    """Rotate the pairs (i, i + D/2) of v [..., D] by the angles whose cos / sin are given as [..., D/2]."""
    v = np.asarray(v, dtype=np.float64)
    half = v.shape[-1] // 2
    a, b = v[..., :half], v[..., half:]
    return np.concatenate([a * cos - b * sin, b * cos + a * sin], axis=-1)


def register_qkv(x, cu_seqlens, idx: np.ndarray, w_norm, w_qkv, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 rope_cos, rope_sin, eps: float = 1e-6):
    """Hidden states x [total, d_model] -> (Q' [B,R,Hq,D], K' [B,R,Hkv,D], V' [B,R,Hkv,D]) of the register rows only:
    gather rows idx[b] of every sequence, RMS-normalise, multiply by W_qkv^T (w_qkv [(Hq+2Hkv)*D, d_model], rows
    ordered Q heads, K heads, V heads), rotate Q and K by the ORIGINAL position idx[b][m] of each register."""
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w_qkv, dtype=np.float64)
    b_, r_ = idx.shape
    q = np.zeros((b_, r_, n_q_heads, head_dim))
    k = np.zeros((b_, r_, n_kv_heads, head_dim))
    v = np.zeros((b_, r_, n_kv_heads, head_dim))
    for b in range(b_):
        for m in range(r_):
            pos = int(idx[b, m])
            y = rms_norm(x[int(cu_seqlens[b]) + pos], w_norm, eps) @ w.T
            qh = y[: n_q_heads * head_dim].reshape(n_q_heads, head_dim)
            kh = y[n_q_heads * head_dim:(n_q_heads + n_kv_heads) * head_dim].reshape(n_kv_heads, head_dim)
            q[b, m] = apply_rope(qh, rope_cos[pos], rope_sin[pos])
            k[b, m] = apply_rope(kh, rope_cos[pos], rope_sin[pos])
            v[b, m] = y[(n_q_heads + n_kv_heads) * head_dim:].reshape(n_kv_heads, head_dim)
    return q, k, v


# --------------------------------------------------------------------------
# Eq. 4 (cache append, then attend over K_{1:t}) with the decode rule of
# Section 3.2: layers l < k see prompt ++ generated, layers l >= k see
# registers ++ generated.
# --------------------------------------------------------------------------
def decode_attention(q_row, keys, values, scale: Optional[float] = None) -> np.ndarray:
    """One query vector against a list of keys/values (no mask: all are past or self).
    q_row [D]; keys, values [n, D] -> [D] float64."""
    q_row = np.asarray(q_row, dtype=np.float64)
    keys = np.asarray(keys, dtype=np.float64)
    values = np.asarray(values, dtype=np.float64)
    s = (keys @ q_row) * _scale(q_row.shape[0], scale)
    p = np.exp(s - np.max(s))
    return (p @ values) / np.sum(p)


class DecodeState:
    """KV cache of ONE layer during decoding, as python lists (Eq. 4).

    shared_k/shared_v: per sequence, the keys every beam of that sequence sees before the
    generated tokens: the whole prompt for a layer l < k, or the compact register rows for
    a layer l >= k ([n_b, Hkv, D] each).  Every beam owns a private list of generated K/V.
    """

    def __init__(self, shared_k: List[np.ndarray], shared_v: List[np.ndarray], beams: int,
                 scale: Optional[float] = None):
        self.shared_k = [np.asarray(x, dtype=np.float64) for x in shared_k]
        self.shared_v = [np.asarray(x, dtype=np.float64) for x in shared_v]
        self.beams = beams
        self.scale = scale
        n = len(shared_k) * beams
        self.priv_k: List[List[np.ndarray]] = [[] for _ in range(n)]
        self.priv_v: List[List[np.ndarray]] = [[] for _ in range(n)]

    def step(self, q, k_new, v_new, parents: Optional[Sequence[int]] = None, rows=None) -> np.ndarray:
        """q [B*W,Hq,D], k_new,v_new [B*W,Hkv,D]; parents[j] in [0,W) = the beam of the same
        sequence whose generated history beam j continues.  Returns O float64 [B*W,Hq,D].
        rows: optional set of (beam, query head) pairs; the cache is updated for every beam but only
        those outputs are computed (the others stay zero) -- for workloads too large to compute in full."""
        w = self.beams
        n = len(self.priv_k)
        if parents is not None:
            pk = [list(self.priv_k[(j // w) * w + int(parents[j])]) for j in range(n)]
            pv = [list(self.priv_v[(j // w) * w + int(parents[j])]) for j in range(n)]
            self.priv_k, self.priv_v = pk, pv
        q = np.asarray(q, dtype=np.float64)
        hq, d = q.shape[1], q.shape[2]
        hkv = k_new.shape[1]
        g = hq // hkv
        out = np.zeros((n, hq, d), dtype=np.float64)
        for j in range(n):
            self.priv_k[j].append(np.asarray(k_new[j], dtype=np.float64))   # Eq. 4: append first,
            self.priv_v[j].append(np.asarray(v_new[j], dtype=np.float64))   # then attend (self included)
            b = j // w
            if rows is not None and not any((j, h) in rows for h in range(hq)):
                continue
            gen_k = np.stack(self.priv_k[j], axis=0)
            gen_v = np.stack(self.priv_v[j], axis=0)
            for h in range(hq):
                if rows is not None and (j, h) not in rows:
                    continue
                keys = np.concatenate([self.shared_k[b][:, h // g, :], gen_k[:, h // g, :]], axis=0)
                vals = np.concatenate([self.shared_v[b][:, h // g, :], gen_v[:, h // g, :]], axis=0)
                out[j, h] = decode_attention(q[j, h], keys, vals, self.scale)
        return out

    def entries(self, b: int) -> int:
        """KV entries one beam of sequence b reads in this layer (per kv head)."""
        return self.shared_k[b].shape[0] + len(self.priv_k[b * self.beams])


# --------------------------------------------------------------------------
# Section 3.2, "Training": the sample is X ++ Y = [R_prefix; Prompt; R_suffix; Y] (Eq. 5-6, Y the target identifier,
# teacher-forced), the loss of Eq. 7 is taken on Y, and the attention differs from ordinary finetuning only in who
# takes part: layers l <= k (1-indexed) all tokens, layers l > k only register and generated (target) tokens.
# Forward is Eq. 3 under that rule; backward is the chain rule through Eq. 3:
#   P = softmax(S), O = P V   =>   dV = P^T dO,  dP = dO V^T,  dS = P o (dP - rowsum(dO o O)),  dQ = dS K c,  dK = dS^T Q c
# with c the logit scale.  Query heads of a group add their dK, dV into the kv head they share.
# --------------------------------------------------------------------------
def participating_indices(seqlens: Sequence[int], r_head: int, r_tail: int, n_target: int) -> np.ndarray:
    """Positions of the tokens that take part in a layer l > k of a TRAINING sequence of length L_b (targets
    included): the r_head prefix registers, the r_tail suffix registers and the n_target target tokens, in order,
    int32 [B, r_head + r_tail + n_target].  The suffix registers and the targets are the last r_tail + n_target rows."""
    return register_indices(seqlens, r_head, r_tail + n_target)


def causal_attention_grad(q, k, v, cu_seqlens, d_o, scale: Optional[float] = None):
    """Gradients of causal_attention's output with respect to q, k, v for an upstream gradient d_o [total,Hq,D]:
    returns (dq [total,Hq,D], dk [total,Hkv,D], dv [total,Hkv,D]), float64."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    d_o = np.asarray(d_o, dtype=np.float64)
    total, hq, d = q.shape
    g = hq // k.shape[1]
    sc = _scale(d, scale)
    dq, dk, dv = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v)
    for b in range(len(cu_seqlens) - 1):
        lo, hi = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        n = hi - lo
        if n == 0:
            continue
        allowed = np.tril(np.ones((n, n), dtype=bool))
        for h in range(hq):
            kh = h // g
            s = np.where(allowed, (q[lo:hi, h, :] @ k[lo:hi, kh, :].T) * sc, -np.inf)
            p, _ = _softmax_rows(s)
            o = p @ v[lo:hi, kh, :]
            go = d_o[lo:hi, h, :]
            dv[lo:hi, kh, :] += p.T @ go
            dp = go @ v[lo:hi, kh, :].T
            ds = p * (dp - np.sum(go * o, axis=1, keepdims=True))
            dq[lo:hi, h, :] = (ds @ k[lo:hi, kh, :]) * sc
            dk[lo:hi, kh, :] += (ds.T @ q[lo:hi, h, :]) * sc
    return dq, dk, dv


def participating_attention(q_p, k_p, v_p, scale: Optional[float] = None):
    """A layer l > k of a training sample on the rows that take part (gathered in order [prefix; suffix; targets]):
    causal attention among them.  q_p [B,P,Hq,D], k_p, v_p [B,P,Hkv,D] -> (O [B,P,Hq,D], LSE [B,Hq,P]) float64."""
    b_, p_, hq, d = q_p.shape
    if p_ == 0:
        return np.zeros((b_, 0, hq, d)), np.zeros((b_, hq, 0))
    cu = np.arange(b_ + 1, dtype=np.int64) * p_
    o, lse = causal_attention(np.asarray(q_p).reshape(b_ * p_, hq, d), np.asarray(k_p).reshape(b_ * p_, -1, d),
                              np.asarray(v_p).reshape(b_ * p_, -1, d), cu, scale)
    return o.reshape(b_, p_, hq, d), lse.reshape(hq, b_, p_).transpose(1, 0, 2).copy()


def participating_attention_grad(q_p, k_p, v_p, d_o_p, scale: Optional[float] = None):
    """Backward of participating_attention: (dq_p, dk_p, dv_p), shapes of the inputs, float64."""
    b_, p_, hq, d = q_p.shape
    hkv = k_p.shape[2]
    if p_ == 0:
        return np.zeros((b_, 0, hq, d)), np.zeros((b_, 0, hkv, d)), np.zeros((b_, 0, hkv, d))
    cu = np.arange(b_ + 1, dtype=np.int64) * p_
    dq, dk, dv = causal_attention_grad(np.asarray(q_p).reshape(b_ * p_, hq, d), np.asarray(k_p).reshape(b_ * p_, hkv, d),
                                       np.asarray(v_p).reshape(b_ * p_, hkv, d), cu,
                                       np.asarray(d_o_p).reshape(b_ * p_, hq, d), scale)
    return dq.reshape(b_, p_, hq, d), dk.reshape(b_, p_, hkv, d), dv.reshape(b_, p_, hkv, d)


# --------------------------------------------------------------------------
# Appendix A.3: item identifiers are generated by beam search (beam size 20).  The paper gives the beam size only; the
# selection rule is that of ordinary beam search: after a step the W continuations (beam, token) with the highest
# cumulative log-probability survive.
# --------------------------------------------------------------------------
def beam_topk(logprobs, beam_scores, beams: int, n_live: Optional[int] = None):
    """logprobs [B*W, V] (log-probability of every token after every beam), beam_scores [B*W] (cumulative
    log-probability of every beam so far) -> (parent int32 [B*W], token int32 [B*W], score float32 [B*W]).

    Candidate (w, v) of a sequence scores beam_scores[w] + logprobs[w, v], the sum taken in float32 (the precision
    the selection is made in; the inputs are float32).  Only beams w < n_live of every sequence offer candidates
    (at the first step all beams hold the same history, so n_live = 1); default: all.  Output slot i of a sequence gets
    the i-th best candidate: higher score first, equal scores in increasing order of the flat candidate index
    w * V + v.  parent is the beam index within the sequence.
    """
    lp = np.asarray(logprobs, dtype=np.float32)
    sc = np.asarray(beam_scores, dtype=np.float32)
    n, vocab = lp.shape
    live = beams if n_live is None else int(n_live)
    if not (1 <= live <= beams) or live * vocab < beams:
        raise ValueError("need at least `beams` candidates per sequence")
    parent = np.zeros(n, dtype=np.int32)
    token = np.zeros(n, dtype=np.int32)
    score = np.zeros(n, dtype=np.float32)
    for b in range(n // beams):
        rows = slice(b * beams, b * beams + live)
        cand = (sc[rows, None] + lp[rows]).astype(np.float32).reshape(-1)       # flat index w * V + v
        order = np.argsort(-cand, kind="stable")[:beams]                          # stable: ties keep index order
        parent[b * beams:(b + 1) * beams] = order // vocab
        token[b * beams:(b + 1) * beams] = order % vocab
        score[b * beams:(b + 1) * beams] = cand[order]
    return parent, token, score


# --------------------------------------------------------------------------
# Section 3.3: Eq. 8 (attention/compute ratio), Eq. 9 (KV-cache ratio), Eq. 13.
# --------------------------------------------------------------------------
def kv_entries(seqlens: Sequence[int], n_layers: int, split_k: int, n_regs: int, generated: int = 0,
               n_kv_heads: int = 1) -> Tuple[int, int]:
    """(EARN entries, vanilla entries): N_KV = n_h (k L + (N-k) r) against n_h N L, each layer also
    holding the generated tokens."""
    earn = vanilla = 0
    for L in seqlens:
        L = int(L)
        for layer in range(n_layers):
            vanilla += L + generated
            earn += (L if layer < split_k else n_regs) + generated
    return earn * n_kv_heads, vanilla * n_kv_heads


def gamma_cache(n_layers: int, split_k: int, prompt_len: int, n_regs: int) -> float:
    """Eq. 9: fraction of the KV cache removed, 1 - (kL + (N-k) r) / (N L)."""
    return 1.0 - (split_k * prompt_len + (n_layers - split_k) * n_regs) / (n_layers * prompt_len)


def layer_flops(length: int, n_heads: int, d_attn: int, d_hidden: int, d_ffn: int) -> float:
    """Eq. 18: FLOPs of one decoder layer over `length` tokens, 4L[n_h d_a (2 d_h + L) + d_h d_f]."""
    return 4.0 * length * (n_heads * d_attn * (2 * d_hidden + length) + d_hidden * d_ffn)


def gamma_attn(n_layers: int, split_k: int, prompt_len: int, n_regs: int, n_heads: int, d_attn: int,
               d_hidden: int, d_ffn: int) -> float:
    """Eq. 8: (k FLOPs_layer(L) + (N-k) FLOPs_layer(r)) / (N FLOPs_layer(L))."""
    full = layer_flops(prompt_len, n_heads, d_attn, d_hidden, d_ffn)
    reg = layer_flops(n_regs, n_heads, d_attn, d_hidden, d_ffn)
    return (split_k * full + (n_layers - split_k) * reg) / (n_layers * full)


def speedup(n_layers: int, split_k: int, prompt_len: int, n_regs: int, n_heads: int, d_attn: int,
            d_hidden: int, d_ffn: int) -> float:
    """Eq. 13 in the compute-bound regime: T_vanilla / T_EARN = 1 / Gamma_attn (about N / k)."""
    return 1.0 / gamma_attn(n_layers, split_k, prompt_len, n_regs, n_heads, d_attn, d_hidden, d_ffn)


# --------------------------------------------------------------------------
# Appendix A.1, Eq. 14-15: attention diagnostics for one row of scores p_1..p_n.
# --------------------------------------------------------------------------
def attention_scores(q_row, keys, scale: Optional[float] = None) -> np.ndarray:
    q_row = np.asarray(q_row, dtype=np.float64)
    s = (np.asarray(keys, dtype=np.float64) @ q_row) * _scale(q_row.shape[0], scale)
    p = np.exp(s - np.max(s))
    return p / np.sum(p)


def sparsity(p: np.ndarray, eps: float = 0.05) -> float:
    """Eq. 14: share of scores above eps."""
    return float(np.mean(p > eps))


def sinks(p: np.ndarray, t_head: int = 3, tail_span: int = 3) -> Tuple[float, float]:
    """Eq. 15 with 1-based positions: Sink_head = sum_{i<=T_h} p_i, Sink_tail = sum_{i>=n-tail_span} p_i."""
    n = len(p)
    return float(np.sum(p[:t_head])), float(np.sum(p[max(n - tail_span - 1, 0):]))
