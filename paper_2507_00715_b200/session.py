"""Call sequencing for one batch: owns the caches and workspace and issues the C-ABI calls in the
order of the hot path (Section 3.2, "Inference").  No arithmetic happens here."""
from __future__ import annotations

from typing import List, Optional

import numpy as np
import torch

from . import binding as B


class EarnSession:
    """One batch of prompts through prefill and decode.

    Layers ``l < split_k`` keep a reference to the caller's packed K/V (read in place during decode);
    layers ``l >= split_k`` own a paged compact register cache.  Every layer owns a private
    (generated-token) cache of ``max_new`` tokens per beam.
    """

    def __init__(self, n_layers: int, split_k: int, n_q_heads: int, n_kv_heads: int, head_dim: int, dtype: torch.dtype,
                 cu_seqlens: np.ndarray, r_head: int, r_tail: int, beams: int = 1, max_new: int = 1,
                 softmax_scale: float = 0.0, device="cuda", paged_shuffle_seed: Optional[int] = None,
                 paged_private_seed: Optional[int] = None):
        self.device = torch.device(device)
        self.dtype = dtype
        self.model = B.make_model(n_layers, split_k, n_q_heads, n_kv_heads, head_dim, dtype, softmax_scale)
        self.batch = B.Batch(cu_seqlens, r_head, r_tail, device=self.device)
        self.beams, self.max_new = beams, max(1, max_new)
        self.n_layers, self.split_k = n_layers, split_k
        self.Hq, self.Hkv, self.D = n_q_heads, n_kv_heads, head_dim
        nb, R = self.batch.batch, r_head + r_tail
        self.R = R
        self.pages_per_seq = max(1, -(-R // B.PAGE_TOKENS))
        self.n_pages = max(1, nb * self.pages_per_seq)
        # an optional scattered page table exercises the paged addressing; None = identity layout
        self.block_table = None
        if paged_shuffle_seed is not None:
            perm = np.random.Generator(np.random.Philox(paged_shuffle_seed)).permutation(self.n_pages)
            self.block_table = torch.from_numpy(perm.astype(np.int32).reshape(nb, self.pages_per_seq)).to(self.device)
        kw = dict(device=self.device, dtype=dtype)
        self.k_shared: List[Optional[torch.Tensor]] = [None] * n_layers
        self.v_shared: List[Optional[torch.Tensor]] = [None] * n_layers
        self.k_full: List[Optional[torch.Tensor]] = [None] * n_layers
        self.v_full: List[Optional[torch.Tensor]] = [None] * n_layers
        self.k_priv, self.v_priv = [], []
        # the private (generated-token) segment: flat slabs, or pages behind a scattered table (one table for all layers)
        self.priv_table, self.priv_pages_per_beam, self.n_priv_pages = None, 0, 0
        if paged_private_seed is not None:
            self.priv_pages_per_beam = -(-self.max_new // B.PAGE_TOKENS)
            self.n_priv_pages = max(1, nb * beams * self.priv_pages_per_beam)
            perm = np.random.Generator(np.random.Philox(paged_private_seed)).permutation(self.n_priv_pages)
            self.priv_table = torch.from_numpy(perm.astype(np.int32).reshape(nb * beams, self.priv_pages_per_beam)).to(self.device)
        for layer in range(n_layers):
            if layer >= split_k:
                self.k_shared[layer] = torch.zeros(self.n_pages, B.PAGE_TOKENS, n_kv_heads, head_dim, **kw)
                self.v_shared[layer] = torch.zeros(self.n_pages, B.PAGE_TOKENS, n_kv_heads, head_dim, **kw)
            if self.priv_table is not None:
                self.k_priv.append(torch.zeros(self.n_priv_pages, B.PAGE_TOKENS, n_kv_heads, head_dim, **kw))
                self.v_priv.append(torch.zeros(self.n_priv_pages, B.PAGE_TOKENS, n_kv_heads, head_dim, **kw))
            else:
                self.k_priv.append(torch.zeros(nb * beams, self.max_new, n_kv_heads, head_dim, **kw))
                self.v_priv.append(torch.zeros(nb * beams, self.max_new, n_kv_heads, head_dim, **kw))
        self.reg_idx = torch.zeros(nb, max(R, 1), dtype=torch.int32, device=self.device)
        self.lineage = [torch.zeros(nb * beams, self.max_new, dtype=torch.int32, device=self.device) for _ in range(2)]
        self.lineage_cur: Optional[int] = None      # None = identity table
        ws_bytes = B.earn_workspace_bytes(self.model, self.batch, beams)
        self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=self.device)
        B.earn_workspace_init(self.workspace)

    # ---- cache descriptors
    def cache(self, layer: int) -> B.EarnCache:
        lin = None if self.lineage_cur is None else self.lineage[self.lineage_cur]
        return B.make_cache(self.k_shared[layer], self.v_shared[layer], self.block_table, self.pages_per_seq,
                            self.n_pages, self.k_priv[layer], self.v_priv[layer], lin, self.beams, self.max_new,
                            self.reg_idx, self.priv_table, self.priv_pages_per_beam, self.n_priv_pages)

    # ---- prefill
    def prefill_layer(self, layer: int, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor,
                      out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                      q_reg: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Layer < k: full causal attention, returns O [total,Hq,D] and keeps k, v for decode.
        Layer >= k: compaction then register attention, returns O' [B,R,Hq,D]."""
        if layer < self.split_k:
            o = out if out is not None else torch.empty_like(q)
            B.earn_prefill_attn(self.model, self.batch, layer, q, k, v, o, lse, self.workspace)
            self.k_full[layer], self.v_full[layer] = k, v
            return o
        nb = self.batch.batch
        if q_reg is None:
            q_reg = torch.empty(nb, self.R, self.Hq, self.D, device=self.device, dtype=self.dtype)
        o = out if out is not None else torch.empty_like(q_reg)
        cache = self.cache(layer)
        B.earn_compact_kv(self.model, self.batch, layer, k, v, cache, q, q_reg)
        B.earn_register_attn(self.model, self.batch, layer, q_reg, cache, o, self.workspace)
        self.last_q_reg = q_reg
        return o

    def register_layer_fused(self, layer: int, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor,
                             out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Layer >= k in one launch: compaction and register attention together (no gathered copy of the queries).
        Returns O' [B,R,Hq,D]; the compact cache and reg_idx are left as prefill_layer leaves them."""
        o = out if out is not None else torch.empty(self.batch.batch, self.R, self.Hq, self.D, device=self.device,
                                                    dtype=self.dtype)
        B.earn_compact_register_attn(self.model, self.batch, layer, q, k, v, self.cache(layer), o, self.workspace)
        return o

    def set_projection(self, d_model: int, max_pos: int, theta: float = 10000.0, rms_eps: float = 1e-6) -> None:
        """Rotary tables (angles pos * theta^(-2i/D), evaluated in double, stored fp32) and the scratch the
        hidden-state form of the register layers needs."""
        inv = theta ** (-torch.arange(0, self.D, 2, dtype=torch.float64) / self.D)
        ang = torch.arange(max_pos, dtype=torch.float64)[:, None] * inv[None, :]
        self.rope_cos = torch.cos(ang).float().to(self.device)
        self.rope_sin = torch.sin(ang).float().to(self.device)
        self.d_model, self.rms_eps = d_model, rms_eps
        self.x_norm = torch.empty(max(self.batch.batch * self.R, 1), d_model, device=self.device, dtype=self.dtype)

    def register_layer_from_hidden(self, layer: int, x: torch.Tensor, w_norm: torch.Tensor, w_qkv: torch.Tensor,
                                   x_is_compact: bool = False, out: Optional[torch.Tensor] = None,
                                   q_reg: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Layer >= k from the hidden states: projection of the register rows into the compact cache, then register
        attention.  Returns O' [B,R,Hq,D]; call set_projection() first."""
        nb = self.batch.batch
        if q_reg is None:
            q_reg = torch.empty(nb, self.R, self.Hq, self.D, device=self.device, dtype=self.dtype)
        o = out if out is not None else torch.empty_like(q_reg)
        cache = self.cache(layer)
        proj = B.make_proj(self.d_model, self.rope_cos, self.rope_sin, self.rms_eps, x_is_compact)
        B.earn_register_qkv(self.model, self.batch, layer, proj, x, w_norm, w_qkv, self.x_norm, cache, q_reg,
                            self.workspace)
        B.earn_register_attn(self.model, self.batch, layer, q_reg, cache, o, self.workspace)
        self.last_q_reg = q_reg
        return o

    # ---- decode
    def begin_step(self, step: int, parents: Optional[torch.Tensor]) -> None:
        """Re-parent the beams before decode step `step` (>= 2); parents: int32 device [B*W]."""
        if parents is None or self.beams == 1 or step < 2:
            return
        nxt = 0 if self.lineage_cur != 0 else 1
        lin_in = None if self.lineage_cur is None else self.lineage[self.lineage_cur]
        B.earn_beam_reparent(self.batch.batch, self.beams, self.max_new, step, parents, lin_in, self.lineage[nxt])
        self.lineage_cur = nxt

    def decode_layer(self, layer: int, step: int, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor,
                     out: Optional[torch.Tensor] = None) -> torch.Tensor:
        o = out if out is not None else torch.empty_like(q)
        B.earn_decode_attn(self.model, self.batch, layer, step, q, k_new, v_new, self.cache(layer), o,
                           self.k_full[layer], self.v_full[layer], self.workspace)
        return o

    def device_status(self) -> int:
        return B.earn_device_status(self.workspace)

    # ---- accounting (Eq. 9 on the actual buffers): KV entries per kv head held after `generated` steps
    def kv_entries(self, generated: int) -> int:
        lens = np.diff(self.batch.cu_host)
        total = 0
        for layer in range(self.n_layers):
            shared = int(lens.sum()) if layer < self.split_k else self.R * len(lens)
            total += shared + len(lens) * self.beams * generated
        return total
