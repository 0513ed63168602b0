"""Seeded synthetic inputs for the EARN attention path.

This module serves both the CUDA path and the CPU oracle and therefore holds
none of the method's arithmetic: it only draws Q/K/V tensors, prompt lengths
and beam parents from a seed.  The shapes follow the five workloads the build
is measured on; the values are i.i.d. N(0,1) with a dual "attention sink"
bias (Section 1, dual attention sinks; Appendix A.1, Eq. 15) so that the
first and last prompt positions attract a large share of the attention mass.

Recipe, per layer and per tensor (fresh generator seeded from
(seed, layer, tensor tag)):

* Q [total, Hq, D], K and V [total, Hkv, D]  ~ N(0,1) in fp32;
* one unit vector u[kv_head] per workload (from the seed alone);
* K[first row of every sequence] += 4 u,  K[last row] += 4 u;
* if ``sink_q_bias``: Q[:, h] += sqrt(D) * u[h // g], which makes the scaled
  logit of every query toward the two sink keys have mean +4;
* the result is rounded once to the workload dtype (bf16 or fp32).

Hidden-state form of the register layers: X ~ N(0,1) [rows, d_model], the
normalisation weight 1 + 0.1 N(0,1), W_qkv ~ N(0, 1/d_model), each rounded once
to the workload dtype.

Decode-step tensors (one new token per beam) are drawn the same way; beam
parents are uniform integers in [0, W).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Tuple

import numpy as np
import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    n_layers: int          # N
    split_k: int           # k : layers [0,k) see every token, [k,N) only registers
    n_q_heads: int         # Hq
    n_kv_heads: int        # Hkv
    head_dim: int          # D
    dtype: str             # "f32" | "bf16"
    prompt_len: int        # uniform prompt length incl. registers; 0 => ragged
    len_lo: int = 0        # ragged: lengths uniform in [len_lo, len_hi]
    len_hi: int = 0
    r_head: int = 1        # prefix registers
    r_tail: int = 1        # suffix registers
    decode_steps: int = 0  # T
    beams: int = 1         # W
    seed: int = 0
    sink_q_bias: bool = True
    lens: Tuple[int, ...] = ()   # explicit prompt lengths (tests); overrides prompt_len / len_lo / len_hi
    hidden: int = 0        # d_model of the hidden-state form of the register layers; 0 => Hq * D

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def n_regs(self) -> int:
        return self.r_head + self.r_tail

    @property
    def d_model(self) -> int:
        return self.hidden if self.hidden > 0 else self.n_q_heads * self.head_dim

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


CONFIGS: Dict[str, Workload] = {
    "tiny": Workload("tiny", batch=1, n_layers=4, split_k=2, n_q_heads=4, n_kv_heads=4, head_dim=64,
                     dtype="f32", prompt_len=256, r_head=4, r_tail=4, decode_steps=8, beams=1, seed=1),
    "1p5b": Workload("1p5b", batch=32, n_layers=28, split_k=4, n_q_heads=12, n_kv_heads=2, head_dim=128,
                     dtype="bf16", prompt_len=512, r_head=8, r_tail=8, decode_steps=16, beams=1, seed=2),
    "7b": Workload("7b", batch=64, n_layers=32, split_k=8, n_q_heads=32, n_kv_heads=8, head_dim=128,
                   dtype="bf16", prompt_len=1024, r_head=16, r_tail=16, decode_steps=20, beams=1, seed=3),
    "long": Workload("long", batch=8, n_layers=32, split_k=8, n_q_heads=32, n_kv_heads=8, head_dim=128,
                     dtype="bf16", prompt_len=4096, r_head=16, r_tail=16, decode_steps=20, beams=1, seed=4),
    "ragged": Workload("ragged", batch=128, n_layers=32, split_k=8, n_q_heads=32, n_kv_heads=8, head_dim=128,
                       dtype="bf16", prompt_len=0, len_lo=128, len_hi=2048, r_head=16, r_tail=16,
                       decode_steps=20, beams=10, seed=5),
}
# The operating points of the paper's own measurements (Section 4 and Appendix A.3: prompts of 50-200 tokens, one
# register per side, beam 20, item identifiers of 4 tokens, split k = 4 on the multi-head backbone at batch 24 and
# k = 7 on the grouped-query backbone at batch 48), as shapes only.  They are extra workloads for tests and
# timing; the benchmark's headline stays the 7B-class configuration.
CONFIGS["paper_mha"] = Workload("paper_mha", batch=24, n_layers=32, split_k=4, n_q_heads=32, n_kv_heads=32, head_dim=128,
                                dtype="bf16", prompt_len=0, len_lo=50, len_hi=200, r_head=1, r_tail=1, decode_steps=4,
                                beams=20, seed=6)
CONFIGS["paper_gqa"] = Workload("paper_gqa", batch=48, n_layers=28, split_k=7, n_q_heads=28, n_kv_heads=4, head_dim=128,
                                dtype="bf16", prompt_len=0, len_lo=50, len_hi=200, r_head=1, r_tail=1, decode_steps=4,
                                beams=20, seed=7)
LONG_SPLIT_SWEEP = (2, 4, 8, 16)

_TAG = {"q": 1, "k": 2, "v": 3, "dq": 4, "dk": 5, "dv": 6, "len": 7, "u": 8, "parent": 9, "x": 10, "wn": 11, "wqkv": 12,
        "logits": 13, "go": 14}


def _seed_for(w: Workload, tag: str, layer: int = 0, step: int = 0) -> int:
    # a plain mixed-radix key; distinct (seed, tag, layer, step) give distinct streams
    return ((w.seed * 16 + _TAG[tag]) * 4096 + layer) * 4096 + step


def seqlens(w: Workload) -> np.ndarray:
    """Prompt length of every sequence, registers included (int32 [batch])."""
    if w.lens:
        return np.asarray(w.lens, dtype=np.int32)
    if w.prompt_len > 0:
        return np.full((w.batch,), w.prompt_len, dtype=np.int32)
    rng = np.random.Generator(np.random.Philox(_seed_for(w, "len")))
    return rng.integers(w.len_lo, w.len_hi + 1, size=w.batch).astype(np.int32)


def cu_seqlens(w: Workload) -> np.ndarray:
    """Exclusive prefix sum of :func:`seqlens` (int32 [batch+1])."""
    out = np.zeros(w.batch + 1, dtype=np.int32)
    np.cumsum(seqlens(w), out=out[1:])
    return out


def sink_direction(w: Workload) -> torch.Tensor:
    """One fp32 unit vector per kv head, [Hkv, D], CPU."""
    g = torch.Generator()
    g.manual_seed(_seed_for(w, "u"))
    u = torch.randn(w.n_kv_heads, w.head_dim, generator=g, dtype=torch.float32)
    return u / u.norm(dim=1, keepdim=True)


def _randn(shape, seed: int, device) -> torch.Tensor:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32)


def layer_qkv(w: Workload, layer: int, device="cpu") -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """Packed prompt tensors of one layer: Q [total,Hq,D], K,V [total,Hkv,D] in the workload dtype."""
    cu = cu_seqlens(w)
    total = int(cu[-1])
    u = sink_direction(w).to(device)
    q = _randn((total, w.n_q_heads, w.head_dim), _seed_for(w, "q", layer), device)
    k = _randn((total, w.n_kv_heads, w.head_dim), _seed_for(w, "k", layer), device)
    v = _randn((total, w.n_kv_heads, w.head_dim), _seed_for(w, "v", layer), device)
    has_rows = cu[1:] > cu[:-1]   # an empty sequence has no first or last row
    first = torch.as_tensor(cu[:-1][has_rows].astype(np.int64), device=device)
    last = torch.as_tensor((cu[1:] - 1)[has_rows].astype(np.int64), device=device)
    k[first] += 4.0 * u
    # a one-token sequence gets the bias once per role, as the recipe states it
    k[last] += 4.0 * u
    if w.sink_q_bias:
        q += math.sqrt(w.head_dim) * u.repeat_interleave(w.group, dim=0)
    dt = w.torch_dtype
    return q.to(dt), k.to(dt), v.to(dt)


def hidden_states(w: Workload, layer: int, device="cpu", compact: bool = False) -> torch.Tensor:
    """Hidden states entering a layer, ~ N(0,1), in the workload dtype: [total, d_model] for every prompt token, or
    (compact) [B*R, d_model] for the register rows alone."""
    rows = w.batch * w.n_regs if compact else int(cu_seqlens(w)[-1])
    return _randn((rows, w.d_model), _seed_for(w, "x", layer, int(compact)), device).to(w.torch_dtype)


def projection_weights(w: Workload, layer: int, device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
    """(w_norm [d_model] ~ 1 + 0.1 N(0,1),  w_qkv [(Hq + 2 Hkv) * D, d_model] ~ N(0, 1/d_model)), workload dtype; the
    rows of w_qkv are ordered Q heads, K heads, V heads."""
    wn = 1.0 + 0.1 * _randn((w.d_model,), _seed_for(w, "wn", layer), device)
    wq = _randn(((w.n_q_heads + 2 * w.n_kv_heads) * w.head_dim, w.d_model), _seed_for(w, "wqkv", layer), device)
    return wn.to(w.torch_dtype), (wq / math.sqrt(w.d_model)).to(w.torch_dtype)


def decode_qkv(w: Workload, layer: int, step: int, device="cpu"):
    """One decode step (1-based): q [B*W,Hq,D], k_new and v_new [B*W,Hkv,D]."""
    rows = w.batch * w.beams
    u = sink_direction(w).to(device)
    q = _randn((rows, w.n_q_heads, w.head_dim), _seed_for(w, "dq", layer, step), device)
    k = _randn((rows, w.n_kv_heads, w.head_dim), _seed_for(w, "dk", layer, step), device)
    v = _randn((rows, w.n_kv_heads, w.head_dim), _seed_for(w, "dv", layer, step), device)
    if w.sink_q_bias:
        q += math.sqrt(w.head_dim) * u.repeat_interleave(w.group, dim=0)
    dt = w.torch_dtype
    return q.to(dt), k.to(dt), v.to(dt)


def beam_parents(w: Workload, step: int) -> np.ndarray:
    """Parent beam (index within the sequence, in [0,W)) of every beam at a decode step (1-based).

    Step 1 has no history to inherit; its parents are the identity.  int32 [B*W].
    """
    if step <= 1 or w.beams == 1:
        return np.tile(np.arange(w.beams, dtype=np.int32), w.batch)
    rng = np.random.Generator(np.random.Philox(_seed_for(w, "parent", 0, step)))
    return rng.integers(0, w.beams, size=w.batch * w.beams).astype(np.int32)


def beam_logprobs(w: Workload, step: int, vocab: int, device="cpu", allowed: int = 0) -> torch.Tensor:
    """Token log-probabilities after every beam at a decode step, fp32 [B*W, vocab]: the log-softmax of logits
    ~ 3 N(0,1) (there is no model here to produce them).  With allowed > 0 only `allowed` tokens per row, drawn from the
    seed, keep a finite value (identifier generation restricted to valid tokens); the rest are -inf."""
    rows = w.batch * w.beams
    logits = 3.0 * _randn((rows, vocab), _seed_for(w, "logits", 0, step), device)
    if allowed > 0:
        g = torch.Generator()
        g.manual_seed(_seed_for(w, "logits", 1, step))
        keep = torch.zeros(rows, vocab, dtype=torch.bool)
        for r in range(rows):
            keep[r, torch.randperm(vocab, generator=g)[:allowed]] = True
        logits = torch.where(keep.to(device), logits, torch.full_like(logits, float("-inf")))
    return torch.log_softmax(logits, dim=-1)


def upstream_grad(w: Workload, layer: int, shape, device="cpu") -> torch.Tensor:
    """Gradient of the loss with respect to an attention output of the given shape, ~ N(0,1), in the workload dtype
    (there is no loss here to produce it)."""
    return _randn(tuple(shape), _seed_for(w, "go", layer), device).to(w.torch_dtype)
