#!/usr/bin/env python
"""Benchmark of the EARN attention hot path on B200.

One "step" = one batch through the whole path: k full-prefill layers, N-k compaction + register
attention layers, then T decode steps over all N layers (compact cache for l >= k, prompt cache for
l < k).  Default workload: the 7B-class GQA configuration.  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 7b] [--impl reference]
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2507_00715_b200 import replicas, workloads as wl  # noqa: E402

METRIC = "EARN attn tokens/s/GPU (prefill+decode, 7B GQA)"
BEAM_VOCAB = 32000   # vocabulary the beam-selection kernel is timed on (the size of the paper's multi-head backbone's)
L2_BYTES = 126 << 20   # B200
UNIT = "tokens/s"


# Datasheet figures of the part, for context beside the measured ones: dense bf16 tensor throughput and the HBM3e
# bandwidth in its round form (the HGX board is specified at 7.7 TB/s).
NOMINAL = dict(tflops=2250.0, hbm_gbs=8000.0)


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        out = dict(hbm_gbs=p["hbm_gbs"], tflops_burst=p["bf16_tflops"], tflops_sustained=p["bf16_tflops_sustained"],
                   source="measured")
    else:
        out = dict(hbm_gbs=6650.0, tflops_burst=1590.0, tflops_sustained=1400.0, source="fallback")
    out.update(nominal_tflops=NOMINAL["tflops"], nominal_hbm_gbs=NOMINAL["hbm_gbs"],
               note="frac = achieved / measured peak (burst for the tensor-bound kernel); frac_nominal = achieved / datasheet")
    return out


KERNEL_SOURCES = {"prefill": "prefill_tc.cu", "compact": "compact.cu", "register": "register_mma.cu", "register_qkv": "register_qkv.cu",
                  "register_layer": "register_mma.cu", "decode_compact": "decode_short.cu", "decode_full": "decode_mma.cu"}


def source_digest(fname: str) -> str:
    """Digest of a kernel's source: the .cu file and every header of csrc/ it includes, directly or through another
    header (a kernel changes with any of them, and with no other file)."""
    import hashlib
    import re
    csrc = os.path.join(ROOT, "paper_2507_00715_b200", "csrc")
    seen, todo = [], [fname]
    while todo:
        name = todo.pop()
        if name in seen or not os.path.exists(os.path.join(csrc, name)):
            continue
        seen.append(name)
        with open(os.path.join(csrc, name)) as f:
            todo += re.findall(r'^\s*#include\s+"([^"]+)"', f.read(), flags=re.M)
    h = hashlib.sha256()
    for name in [fname] + sorted(n for n in seen if n != fname):
        with open(os.path.join(csrc, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:12]


def read_traffic(name: str) -> dict:
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures summarised in
    profiles/ncu_traffic.txt (lines: workload kind bytes source-file digest).  A figure is dropped when the
    kernel's source file no longer matches the digest recorded with it."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.txt")
    out = {}
    if not os.path.exists(path):
        return out
    with open(path) as f:
        for line in f:
            parts = line.split("#")[0].split()
            if len(parts) != 5 or parts[0] != name:
                continue
            _, kind, nbytes, fname, digest = parts
            if source_digest(fname) == digest:
                out[kind] = float(nbytes)
    return out


def workload_desc(w: wl.Workload) -> str:
    lens = wl.seqlens(w)
    return (f"{w.name}: B={w.batch} N={w.n_layers} k={w.split_k} Hq/Hkv/D={w.n_q_heads}/{w.n_kv_heads}/{w.head_dim} "
            f"{w.dtype} L={int(lens.min())}..{int(lens.max())} (sum {int(lens.sum())}) regs={w.r_head}+{w.r_tail} "
            f"T={w.decode_steps} W={w.beams} seed={w.seed}")


# ------------------------------------------------------------------------------------------------
# algorithmic work (per launch) of each step of the path
# ------------------------------------------------------------------------------------------------
def algorithmic(w: wl.Workload):
    lens = wl.seqlens(w).astype(np.int64)
    es = 4 if w.dtype == "f32" else 2
    D, Hq, Hkv, B, R, W = w.head_dim, w.n_q_heads, w.n_kv_heads, w.batch, w.n_regs, w.beams
    tot = int(lens.sum())
    out = {}
    out["prefill"] = dict(flops=4.0 * D * Hq * float((lens * (lens + 1) // 2).sum()),
                          bytes=float(tot * D * es * (2 * Hq + 2 * Hkv)))
    # compaction: the K and V register rows, read and written, plus the index list.  The gathered Q rows that
    # earn_compact_kv can also write are this library's way of feeding earn_register_attn, not work the method asks
    # for: they count as traffic, not as algorithmic bytes (the register layer's Q rows are counted once, below).
    out["compact"] = dict(flops=0.0, bytes=float(2 * 2 * B * R * Hkv * D * es + B * R * 4))
    out["register"] = dict(flops=4.0 * D * Hq * B * R * (R + 1) / 2, bytes=float(B * R * D * es * (2 * Hq + 2 * Hkv)))
    # hidden-state form of a register layer: the projection of the B*R register rows (bf16 path only)
    M, N, K = B * R, (Hq + 2 * Hkv) * D, w.d_model
    out["register_qkv"] = dict(flops=2.0 * M * N * K, bytes=float(es * (3 * M * K + N * K + M * N + K)))
    s = w.decode_steps   # last step: the longest cache
    qo = 2 * B * W * Hq * D * es + 4 * B * W * Hkv * D * es
    out["decode_compact"] = dict(flops=4.0 * D * Hq * B * W * (R + s), bytes=float(2 * B * (R + W * s) * Hkv * D * es + qo))
    out["decode_full"] = dict(flops=4.0 * D * Hq * W * (tot + B * s), bytes=float(2 * (tot + B * W * s) * Hkv * D * es + qo))
    out["compact_register"] = dict(flops=out["register"]["flops"], bytes=out["compact"]["bytes"] + out["register"]["bytes"])
    out["train_fwd"] = dict(flops=out["prefill"]["flops"], bytes=out["prefill"]["bytes"] + 4.0 * Hq * tot)
    # backward: five products of the forward's two (S, dP, dV, dK, dQ); reads Q, K, V, O, dO, writes dQ, dK, dV
    out["train_bwd"] = dict(flops=2.5 * out["prefill"]["flops"], bytes=float(tot * D * es * (4 * Hq + 4 * Hkv)))
    out["beam_topk"] = dict(flops=0.0, bytes=float(B * W * BEAM_VOCAB * 4 + B * W * 16))
    return out


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device: int):
        self.proc = None
        ident = str(device)
        try:
            uuid = str(torch.cuda.get_device_properties(device).uuid)
            ident = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
        except Exception:
            pass
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", ident, f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return None
        time.sleep(0.15)
        self.proc.terminate()
        try:
            text, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            return None
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in text.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return None
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
# the GPU arm
# ------------------------------------------------------------------------------------------------
class GpuJob:
    def __init__(self, w: wl.Workload, device):
        from paper_2507_00715_b200 import binding as B
        from paper_2507_00715_b200.session import EarnSession
        self.B = B
        self.w = w
        self.dev = device
        self.ses = EarnSession(w.n_layers, w.split_k, w.n_q_heads, w.n_kv_heads, w.head_dim, w.torch_dtype,
                               wl.cu_seqlens(w), w.r_head, w.r_tail, beams=w.beams, max_new=max(w.decode_steps, 1),
                               device=device)
        self.qkv = [wl.layer_qkv(w, layer, device) for layer in range(w.n_layers)]
        self.dec = [[wl.decode_qkv(w, layer, s, device) for layer in range(w.n_layers)]
                    for s in range(1, w.decode_steps + 1)]
        self.parents = [None] + [torch.from_numpy(wl.beam_parents(w, s)).to(device) if w.beams > 1 else None
                                 for s in range(2, w.decode_steps + 1)]
        total = int(wl.cu_seqlens(w)[-1])
        kw = dict(device=device, dtype=w.torch_dtype)
        self.o_full = torch.empty(total, w.n_q_heads, w.head_dim, **kw)
        self.q_reg = torch.empty(w.batch, w.n_regs, w.n_q_heads, w.head_dim, **kw)
        self.o_reg = torch.empty_like(self.q_reg)
        self.o_dec = torch.empty(w.batch * w.beams, w.n_q_heads, w.head_dim, **kw)
        self.fused_register = w.dtype == "bf16" and 0 < w.n_regs <= 128
        self.graphs = None
        self.marks = []

    def device_status(self) -> int:
        return self.ses.device_status()

    def kv_entries(self, generated: int) -> int:
        return self.ses.kv_entries(generated)

    # ---- the step as an ordered list of segments; each segment = consecutive launches of one kind
    def segments(self):
        """[(kind, n_launches, callable)] in the order of the hot path.  `n_launches` counts the calls the
        roofline is quoted per: prefill / decode calls, or (compaction + register attention) pairs."""
        w, ses = self.w, self.ses
        early, late = list(range(w.split_k)), list(range(w.split_k, w.n_layers))
        segs = []
        if early:
            segs.append(("prefill", len(early),
                         lambda: [ses.prefill_layer(l, *self.qkv[l], out=self.o_full) for l in early]))
        if late:
            # register layers: compaction + register attention, in one launch where the library has the fused kernel
            # (bf16, at most 128 registers), through the two calls otherwise
            if self.fused_register:
                segs.append(("register_layer", len(late),
                             lambda: [ses.register_layer_fused(l, *self.qkv[l], out=self.o_reg) for l in late]))
            else:
                segs.append(("register_layer", len(late),
                             lambda: [ses.prefill_layer(l, *self.qkv[l], out=self.o_reg, q_reg=self.q_reg) for l in late]))
        for s in range(1, w.decode_steps + 1):
            if early:
                def f(s=s):
                    ses.begin_step(s, self.parents[s - 1])
                    for l in early:
                        ses.decode_layer(l, s, *self.dec[s - 1][l], out=self.o_dec)
                segs.append(("decode_full", len(early), f))
            if late:
                def f2(s=s, first=not early):
                    if first:
                        ses.begin_step(s, self.parents[s - 1])
                    for l in late:
                        ses.decode_layer(l, s, *self.dec[s - 1][l], out=self.o_dec)
                segs.append(("decode_compact", len(late), f2))
        return segs

    def capture_graphs(self):
        """One CUDA graph per segment (the launches of a step never change between steps)."""
        self.ses.lineage_cur = None
        self.graphs = []
        for kind, n, fn in self.segments():
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                fn()
            self.graphs.append((kind, n, g))
        torch.cuda.synchronize()

    def step(self, record=False):
        """One pass of the whole hot path.  With record=True an event is recorded at every segment
        boundary so that each kind of launch gets a live duration inside the timed region."""
        self.ses.lineage_cur = None
        items = self.graphs if self.graphs is not None else self.segments()
        marks = []
        for kind, n, g in items:
            if record:
                e = torch.cuda.Event(enable_timing=True)
                e.record()
                marks.append((kind, n, e))
            if self.graphs is not None:
                g.replay()
            else:
                g()
        if record:
            e = torch.cuda.Event(enable_timing=True)
            e.record()
            marks.append((None, 0, e))
            self.marks.append(marks)

    def segment_times(self):
        """{kind: (seconds per launch, launches per step, share of step time)} from the recorded events."""
        tot, cnt, steps = {}, {}, len(self.marks)
        for marks in self.marks:
            for (kind, n, e0), (_, _, e1) in zip(marks[:-1], marks[1:]):
                tot[kind] = tot.get(kind, 0.0) + e0.elapsed_time(e1) * 1e-3
                cnt[kind] = cnt.get(kind, 0) + n
        whole = sum(tot.values())
        return {k: (tot[k] / cnt[k], cnt[k] // steps, tot[k] / whole) for k in tot}

    # ---- per-kernel timing in isolation (explains the step time; not the headline)
    def time_parts(self, reps=3):
        w, ses = self.w, self.ses
        res = {}

        def timed(fn, n_launch):
            fn()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                fn()
            g.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                g.replay()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) * 1e-3 / (reps * n_launch)

        early = list(range(w.split_k))
        late = list(range(w.split_k, w.n_layers))
        if early:
            res["prefill"] = timed(lambda: [ses.prefill_layer(l, *self.qkv[l], out=self.o_full) for l in early], len(early))
        if late:
            caches = {l: ses.cache(l) for l in late}
            res["compact"] = timed(lambda: [self.B.earn_compact_kv(ses.model, ses.batch, l, self.qkv[l][1], self.qkv[l][2],
                                                                   caches[l], self.qkv[l][0], self.q_reg) for l in late], len(late))
            res["register"] = timed(lambda: [self.B.earn_register_attn(ses.model, ses.batch, l, self.q_reg, caches[l],
                                                                       self.o_reg, ses.workspace) for l in late], len(late))
            if self.fused_register:
                res["compact_register"] = timed(lambda: [ses.register_layer_fused(l, *self.qkv[l], out=self.o_reg) for l in late], len(late))
            if w.dtype == "bf16" and w.head_dim == 128 and w.n_regs > 0:
                # the same layers from hidden states (not part of the timed step, whose inputs are Q, K, V): one x for
                # every layer, weights per layer so that they come from HBM as they would in a model
                ses.set_projection(w.d_model, int(wl.seqlens(w).max()))
                x = wl.hidden_states(w, late[0], self.dev)
                wts = [wl.projection_weights(w, l, self.dev) for l in late]
                proj = self.B.make_proj(w.d_model, ses.rope_cos, ses.rope_sin)
                res["register_qkv"] = timed(lambda: [self.B.earn_register_qkv(ses.model, ses.batch, l, proj, x, wts[i][0], wts[i][1],
                                                                              ses.x_norm, caches[l], self.q_reg, ses.workspace)
                                                     for i, l in enumerate(late)], len(late))
                del x, wts
        if early and w.dtype == "bf16":
            # training-time attention of one full layer (Section 3.2 "Training"; not part of the timed inference step):
            # forward with LSE, then backward (dQ, dK, dV); useful flops: forward 4 D per causal pair and head, backward 2.5 x
            q, k, v = self.qkv[0]
            total = q.shape[0]
            tws = torch.empty(self.B.earn_train_workspace_bytes(ses.model, ses.batch), dtype=torch.uint8, device=self.dev)
            self.B.earn_workspace_init(tws)
            lse = torch.empty(w.n_q_heads, total, dtype=torch.float32, device=self.dev)
            d_o = wl.upstream_grad(w, 0, q.shape, self.dev)
            dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
            res["train_fwd"] = timed(lambda: self.B.earn_train_attn_fwd(ses.model, ses.batch, 0, 0, q, k, v, self.o_full, lse, tws), 1)
            res["train_bwd"] = timed(lambda: self.B.earn_train_attn_bwd(ses.model, ses.batch, 0, 0, q, k, v, self.o_full, lse, d_o,
                                                                        dq, dk, dv, tws), 1)
            del tws, lse, d_o, dq, dk, dv
        if w.beams > 1:
            # beam selection between decode steps (not part of the timed step, which has no output layer to produce
            # log-probabilities): every log-probability read once, B * W * V * 4 bytes
            vocab = BEAM_VOCAB
            rows = w.batch * w.beams
            # several inputs in turn, together larger than L2 (one of them may fit in it)
            n_in = max(2, min(8, -(-(3 * L2_BYTES) // (rows * vocab * 4))))
            lps = [wl.beam_logprobs(w, 1 + i, vocab, self.dev) for i in range(n_in)]
            sc = [torch.zeros(rows, device=self.dev), torch.zeros(rows, device=self.dev)]
            par, tok = (torch.zeros(rows, dtype=torch.int32, device=self.dev) for _ in range(2))
            ws = torch.empty(self.B.earn_beam_topk_workspace_bytes(w.batch, w.beams, vocab), dtype=torch.uint8, device=self.dev)
            res["beam_topk"] = timed(lambda: [self.B.earn_beam_topk(w.batch, w.beams, w.beams, vocab, lp, sc[0], par, tok, sc[1], ws)
                                              for lp in lps], n_in)
            del lps, ws
        if w.decode_steps > 0:
            s = w.decode_steps
            if late:
                res["decode_compact"] = timed(lambda: [ses.decode_layer(l, s, *self.dec[s - 1][l], out=self.o_dec) for l in late], len(late))
            if early:
                res["decode_full"] = timed(lambda: [ses.decode_layer(l, s, *self.dec[s - 1][l], out=self.o_dec) for l in early], len(early))
        return res

    # ---- end-to-end: inputs start in pinned host memory, outputs end there
    def setup_e2e(self):
        def pin(t):
            return torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t)
        self.h_qkv = [tuple(pin(t) for t in trip) for trip in self.qkv]
        self.h_dec = [[tuple(pin(t) for t in trip) for trip in row] for row in self.dec]
        w = self.w
        self.h_o_full = [torch.empty(self.o_full.shape, dtype=self.o_full.dtype, pin_memory=True) for _ in range(w.split_k)]
        self.h_o_reg = [torch.empty(self.o_reg.shape, dtype=self.o_reg.dtype, pin_memory=True)
                        for _ in range(w.n_layers - w.split_k)]
        self.h_o_dec = torch.empty((max(w.decode_steps, 1), w.n_layers) + tuple(self.o_dec.shape), dtype=self.o_dec.dtype,
                                   pin_memory=True)
        nbytes = lambda t: t.numel() * t.element_size()   # noqa: E731
        h2d = sum(nbytes(t) for trip in self.h_qkv for t in trip) + sum(nbytes(t) for row in self.h_dec for trip in row for t in trip)
        d2h = sum(nbytes(t) for t in self.h_o_full) + sum(nbytes(t) for t in self.h_o_reg)
        d2h += w.decode_steps * w.n_layers * nbytes(self.o_dec)
        return h2d, d2h

    def step_e2e(self):
        """One pass with every input starting in pinned host memory and every output ending there.  Prefill moves
        26 GB in and 5 GB out at the 7B shapes, so its copies run on their own streams: the inputs of layer l+1
        arrive while layer l computes, outputs drain behind it (two output buffers alternate).  The decode copies
        are small and stay on the compute stream."""
        w, ses = self.w, self.ses
        ses.lineage_cur = None
        cs = torch.cuda.current_stream()
        if not hasattr(self, "s_h2d"):
            self.s_h2d, self.s_d2h = torch.cuda.Stream(), torch.cuda.Stream()
            self.o_full_alt, self.o_reg_alt = torch.empty_like(self.o_full), torch.empty_like(self.o_reg)
        start = torch.cuda.Event()
        start.record(cs)                      # the previous pass still reads the device inputs (decode reads K/V in place)
        self.s_h2d.wait_event(start)
        arrived = []
        with torch.cuda.stream(self.s_h2d):
            for layer in range(w.n_layers):
                for d, h in zip(self.qkv[layer], self.h_qkv[layer]):
                    d.copy_(h, non_blocking=True)
                e = torch.cuda.Event()
                e.record(self.s_h2d)
                arrived.append(e)
        drained = {}                          # output buffer id -> event after which it may be overwritten
        last = None
        for layer in range(w.n_layers):
            cs.wait_event(arrived[layer])
            q, k, v = self.qkv[layer]
            full = layer < w.split_k
            out = (self.o_full, self.o_full_alt)[layer & 1] if full else (self.o_reg, self.o_reg_alt)[layer & 1]
            if id(out) in drained:
                cs.wait_event(drained[id(out)])
            if full:
                ses.prefill_layer(layer, q, k, v, out=out)
                host = self.h_o_full[layer]
            else:
                if self.fused_register:
                    ses.register_layer_fused(layer, q, k, v, out=out)
                else:
                    ses.prefill_layer(layer, q, k, v, out=out, q_reg=self.q_reg)
                host = self.h_o_reg[layer - w.split_k]
            done = torch.cuda.Event()
            done.record(cs)
            self.s_d2h.wait_event(done)
            with torch.cuda.stream(self.s_d2h):
                host.copy_(out, non_blocking=True)
                last = torch.cuda.Event()
                last.record(self.s_d2h)
            drained[id(out)] = last
        for s in range(1, w.decode_steps + 1):
            ses.begin_step(s, self.parents[s - 1])
            for layer in range(w.n_layers):
                for d, h in zip(self.dec[s - 1][layer], self.h_dec[s - 1][layer]):
                    d.copy_(h, non_blocking=True)
                q, k, v = self.dec[s - 1][layer]
                ses.decode_layer(layer, s, q, k, v, out=self.o_dec)
                self.h_o_dec[s - 1, layer].copy_(self.o_dec, non_blocking=True)
        if last is not None:
            cs.wait_event(last)               # the pass ends when its last output has reached the host


# ------------------------------------------------------------------------------------------------
# the CPU oracle arm (a baseline, not a target): one sequence of the workload through every layer and step
# ------------------------------------------------------------------------------------------------
class OracleSample:
    def __init__(self, w: wl.Workload, job: GpuJob | None, layer_stride: int = 1):
        """One sequence of the workload through every `layer_stride`-th layer (all decode steps); with a stride the
        measured time is scaled back by it, which keeps the full/register layer mix when the stride divides k and N."""
        if layer_stride > 1 and (w.split_k % layer_stride or w.n_layers % layer_stride):
            layer_stride = 1
        self.stride = layer_stride
        lens = wl.seqlens(w)
        cu = wl.cu_seqlens(w)
        self.w1 = w.replace(batch=1, lens=(int(lens[0]),))
        f = lambda t: t.detach().float().cpu().numpy()   # noqa: E731
        if job is not None:       # the same tensors the GPU arm uses
            self.qkv = [tuple(f(t[cu[0]:cu[1]]) for t in trip) for trip in job.qkv]
            self.dec = [[tuple(f(t[:w.beams]) for t in trip) for trip in row] for row in job.dec]
        else:                     # no device: draw the one-sequence workload on the host
            dev = "cuda" if torch.cuda.is_available() else "cpu"
            every = lambda l, fn: fn() if l % layer_stride == 0 else None   # noqa: E731
            self.qkv = [every(l, lambda: tuple(f(t) for t in wl.layer_qkv(self.w1, l, dev))) for l in range(w.n_layers)]
            self.dec = [[every(l, lambda: tuple(f(t) for t in wl.decode_qkv(self.w1, l, s, dev))) for l in range(w.n_layers)]
                        for s in range(1, w.decode_steps + 1)]
        self.parents = [None] + [wl.beam_parents(w, s)[:w.beams] if w.beams > 1 else None
                                 for s in range(2, w.decode_steps + 1)]
        self.tokens = int(lens[0]) + w.beams * w.decode_steps
        layers = f"all {w.n_layers} layers" if layer_stride == 1 else \
            f"every {layer_stride}th of the {w.n_layers} layers (time scaled by {layer_stride})"
        self.desc = (f"sequence 0 of {w.batch} (L={int(lens[0])}, {w.beams} beam(s)): {layers} of prefill "
                     f"and all {w.decode_steps} decode steps")

    def run(self) -> float:
        from oracle import earn_oracle as orc
        w = self.w1
        t0 = time.perf_counter()
        cu = np.array([0, w.lens[0]])
        idx = orc.register_indices(w.lens, w.r_head, w.r_tail)
        states = {}
        layers = range(0, w.n_layers, self.stride)
        for layer in layers:
            q, k, v = self.qkv[layer]
            if layer < w.split_k:
                orc.causal_attention(q, k, v, cu)
                states[layer] = orc.DecodeState([k], [v], w.beams)
            else:
                kc, vc, qc = orc.compact(k, cu, idx), orc.compact(v, cu, idx), orc.compact(q, cu, idx)
                orc.register_attention(qc, kc, vc)
                states[layer] = orc.DecodeState([kc[0]], [vc[0]], w.beams)
        for s in range(1, w.decode_steps + 1):
            for layer in layers:
                q, k, v = self.dec[s - 1][layer]
                states[layer].step(q, k, v, self.parents[s - 1])
        return (time.perf_counter() - t0) * self.stride


def profile_one_kernel(w: wl.Workload, dev, which: str, launches: int = 3):
    """One layer of the workload, one kind of launch, `launches` times (a few GB at most on the device)."""
    early = which in ("prefill", "decode_full", "train_bwd")
    # keep the layer on the side of the split the kernel belongs to; one full layer + one register layer
    w1 = w.replace(n_layers=2, split_k=1)
    layer = 0 if early else 1
    job = GpuJob.__new__(GpuJob)
    from paper_2507_00715_b200 import binding as B
    from paper_2507_00715_b200.session import EarnSession
    ses = EarnSession(w1.n_layers, w1.split_k, w1.n_q_heads, w1.n_kv_heads, w1.head_dim, w1.torch_dtype,
                      wl.cu_seqlens(w1), w1.r_head, w1.r_tail, beams=w1.beams, max_new=max(w1.decode_steps, 1), device=dev)
    q, k, v = wl.layer_qkv(w1, layer, dev)
    o = torch.empty_like(q)
    q_reg = torch.empty(w1.batch, w1.n_regs, w1.n_q_heads, w1.head_dim, device=dev, dtype=w1.torch_dtype)
    o_reg = torch.empty_like(q_reg)
    s_last = max(w1.decode_steps, 1)
    dq, dk, dv = wl.decode_qkv(w1, layer, s_last, dev)
    o_dec = torch.empty_like(dq)
    if early:
        ses.prefill_layer(0, q, k, v, out=o)            # also registers the prompt K/V for decode
    else:
        ses.prefill_layer(1, q, k, v, out=o_reg, q_reg=q_reg)
    if which == "register_qkv":
        ses.set_projection(w1.d_model, int(wl.seqlens(w1).max()))
        x = wl.hidden_states(w1, 1, dev)
        w_norm, w_qkv = wl.projection_weights(w1, 1, dev)
        proj = B.make_proj(w1.d_model, ses.rope_cos, ses.rope_sin)
    if which == "train_bwd":
        tws = torch.empty(B.earn_train_workspace_bytes(ses.model, ses.batch), dtype=torch.uint8, device=dev)
        B.earn_workspace_init(tws)
        lse = torch.empty(w1.n_q_heads, q.shape[0], dtype=torch.float32, device=dev)
        d_o = wl.upstream_grad(w1, 0, q.shape, dev)
        g_q, g_k, g_v = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
        B.earn_train_attn_fwd(ses.model, ses.batch, 0, 0, q, k, v, o, lse, tws)
    if which == "beam_topk":
        rows = w1.batch * w1.beams
        lp = wl.beam_logprobs(w1, 1, BEAM_VOCAB, dev)
        sc = [torch.zeros(rows, device=dev), torch.zeros(rows, device=dev)]
        par, tok = (torch.zeros(rows, dtype=torch.int32, device=dev) for _ in range(2))
        bws = torch.empty(B.earn_beam_topk_workspace_bytes(w1.batch, w1.beams, BEAM_VOCAB), dtype=torch.uint8, device=dev)
    torch.cuda.synchronize()
    for _ in range(launches):
        if which == "train_bwd":
            B.earn_train_attn_bwd(ses.model, ses.batch, 0, 0, q, k, v, o, lse, d_o, g_q, g_k, g_v, tws)
        elif which == "beam_topk":
            B.earn_beam_topk(w1.batch, w1.beams, w1.beams, BEAM_VOCAB, lp, sc[0], par, tok, sc[1], bws)
        elif which == "prefill":
            ses.prefill_layer(0, q, k, v, out=o)
        elif which == "compact":
            B.earn_compact_kv(ses.model, ses.batch, 1, k, v, ses.cache(1), q, q_reg)
        elif which == "register":
            B.earn_register_attn(ses.model, ses.batch, 1, q_reg, ses.cache(1), o_reg, ses.workspace)
        elif which == "register_layer":
            ses.register_layer_fused(1, q, k, v, out=o_reg)
        elif which == "register_qkv":
            B.earn_register_qkv(ses.model, ses.batch, 1, proj, x, w_norm, w_qkv, ses.x_norm, ses.cache(1), q_reg, ses.workspace)
        else:
            ses.decode_layer(layer, s_last, dq, dk, dv, out=o_dec)
    torch.cuda.synchronize()
    assert ses.device_status() == 0
    print(json.dumps({"profiled": which, "workload": workload_desc(w1), "launches": launches}))


def sweep_split_layer(w: wl.Workload, dev, ks, args):
    """The k sweep of the long-history workload (and of any other): the whole hot path timed once per split layer.
    Section 3.3 predicts time ~ k/N of the vanilla model for prefill (Eq. 8) and a cache of kL + (N-k)r entries
    (Eq. 9); k = N is the vanilla model.  One JSON line per k."""
    lens = wl.seqlens(w)
    tokens = int(lens.sum()) + w.batch * w.beams * w.decode_steps
    base = None
    for k in ks:
        wk = w.replace(split_k=k)
        job = GpuJob(wk, dev)
        job.step()
        torch.cuda.synchronize()
        if not args.no_graphs:
            job.capture_graphs()
        for _ in range(args.warmup):
            job.step()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            job.step(record=True)
        e1.record()
        torch.cuda.synchronize()
        assert job.ses.device_status() == 0
        t = e0.elapsed_time(e1) * 1e-3 / args.steps
        seg = {kind: sec * n * 1e3 for kind, (sec, n, _) in job.segment_times().items()}
        T, N = wk.decode_steps, wk.n_layers
        earn_e, van_e = job.ses.kv_entries(T), N * (int(lens.sum()) + wk.batch * wk.beams * T)
        L, r = float(lens.mean()), wk.n_regs
        line = {"sweep": "split_k", "workload": workload_desc(wk), "k": k, "value": tokens / t, "unit": UNIT,
                "ms_per_step": t * 1e3, "prefill_ms": seg.get("prefill", 0.0) + seg.get("register_layer", 0.0),
                "decode_ms": seg.get("decode_full", 0.0) + seg.get("decode_compact", 0.0),
                "kv_reduction_measured": 1.0 - earn_e / van_e,
                "gamma_cache_eq9": (N - k) * (L - r) / (N * L), "k_over_N": k / N}
        if k == N:
            base = t
        if base is not None:
            line["speedup_vs_vanilla"] = base / t
        print(json.dumps(line), flush=True)
        del job
        torch.cuda.empty_cache()


def blas_threads() -> int:
    try:
        import threadpoolctl
        return max([p["num_threads"] for p in threadpoolctl.threadpool_info() if p.get("user_api") == "blas"] or [1])
    except Exception:
        return os.cpu_count() or 1


def timed_oracle(sample: "OracleSample"):
    """(wall seconds, cores the run kept busy, threads it could have used).  The oracle is numpy: its matrix
    products go to a threaded BLAS, everything else runs on one thread, so the cores it really used are read off
    the process's CPU time over the wall time of the run rather than off the BLAS pool size."""
    c0, w0 = time.process_time(), time.perf_counter()
    t = sample.run()
    c1, w1 = time.process_time(), time.perf_counter()
    busy = (c1 - c0) / max(w1 - w0, 1e-9)
    return t, max(1, int(round(busy))), busy, blas_threads()


# ------------------------------------------------------------------------------------------------
# timers: the GPU arm times with CUDA events on the launching stream; a CPU job (the launcher's test) with the
# host clock
# ------------------------------------------------------------------------------------------------
class DeviceTimer:
    def start(self):
        self.e0, self.e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.e0.record()

    def stop(self):
        self.e1.record()

    def seconds(self) -> float:
        torch.cuda.synchronize()
        return self.e0.elapsed_time(self.e1) * 1e-3


class HostTimer:
    def start(self):
        self.t0 = time.perf_counter()

    def stop(self):
        self.t1 = time.perf_counter()

    def seconds(self) -> float:
        return self.t1 - self.t0


def free_port() -> int:
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        return sock.getsockname()[1]


def _rank_entry(local_rank: int, world: int, port: int, argv, backend: str, job_factory):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(local_rank), LOCAL_RANK=str(local_rank),
                      WORLD_SIZE=str(world))
    main(argv, backend=backend, job_factory=job_factory)


def spawn_ranks(n: int, argv, backend: str = "nccl", job_factory=None) -> None:
    """`bench.py --gpus N` started as ONE process: start N ranks of this program on this node, one per GPU (rank =
    local rank = device index), rendezvous on 127.0.0.1, and wait for them.  Rank 0 prints the line."""
    import torch.multiprocessing as mp
    mp.spawn(_rank_entry, args=(n, free_port(), list(argv), backend, job_factory), nprocs=n, join=True)


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="7b", choices=sorted(wl.CONFIGS))
    ap.add_argument("--split-k", type=int, default=None)
    ap.add_argument("--prompt-len", type=int, default=None, help="override the workload's prompt length (uniform)")
    ap.add_argument("--batch", type=int, default=None, help="override the workload's batch size")
    ap.add_argument("--decode-steps", type=int, default=None,
                    help="override the workload's decode steps T; 0 = the prefill-only operating point")
    ap.add_argument("--impl", default="earn", choices=["earn", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-parts", action="store_true")
    ap.add_argument("--no-graphs", action="store_true", help="plain launches instead of CUDA-graph replay")
    ap.add_argument("--profile-kernel", default=None,
                    choices=["prefill", "compact", "register", "register_layer", "register_qkv", "decode_compact", "decode_full",
                             "train_bwd", "beam_topk"],
                    help="small case for a profiler: allocate ONE layer of the workload and launch that step 3 times")
    ap.add_argument("--sweep-k", default=None,
                    help="comma-separated split layers k: time the workload once per k (one JSON line each, k = N is the "
                         "vanilla model) instead of the single benchmark line")
    args = ap.parse_args(argv)
    args.warmup = max(args.warmup, 3) if args.impl == "earn" else args.warmup
    return args


def pick_workload(args) -> wl.Workload:
    w = wl.CONFIGS[args.config]
    if args.split_k is not None:
        w = w.replace(split_k=args.split_k)
    if args.prompt_len is not None:
        w = w.replace(prompt_len=args.prompt_len, lens=())
    if args.batch is not None:
        w = w.replace(batch=args.batch)
    if args.decode_steps is not None:
        w = w.replace(decode_steps=args.decode_steps)
    return w


def reference_arm(args, w, config):
    sample = OracleSample(w, None, layer_stride=4)   # about a second of oracle work per step
    for _ in range(args.warmup):
        sample.run()
    runs = [timed_oracle(sample) for _ in range(args.steps)]
    t = sum(r[0] for r in runs) / len(runs)
    val = sample.tokens / t
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": config,
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": max(r[1] for r in runs), "kind": "oracle (numpy float64)",
                         "sample": sample.desc, "cores_busy_mean": sum(r[2] for r in runs) / len(runs),
                         "blas_threads_available": runs[0][3]},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


# ------------------------------------------------------------------------------------------------
def main(argv=None, backend: str = "nccl", job_factory=None):
    """One rank of the benchmark (or, for `--gpus N` without a launcher's environment, the parent that starts N).
    job_factory(workload, device, rank) replaces the GPU job -- the launcher's CPU test passes a stand-in that
    has no kernels to run; the rank logic (rendezvous, barrier, max over ranks, rank 0 prints) is the same."""
    args = parse_args(argv)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "earn":
        spawn_ranks(args.gpus, sys.argv[1:] if argv is None else argv, backend, job_factory)
        return

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    w = pick_workload(args)
    lens = wl.seqlens(w)
    tokens_per_step = int(lens.sum()) + w.batch * w.beams * w.decode_steps
    config = {"workload": workload_desc(w), "l2": "per-layer inputs and caches exceed the 126 MB L2; no flush needed",
              "sharding": "every rank runs the whole batch of its own seed (no data-path collective)"}

    if args.impl == "reference":
        if rank == 0:
            reference_arm(args, w, config)
        return

    on_gpu = job_factory is None
    if on_gpu:
        assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
        torch.cuda.set_device(local_rank)
        dev = torch.device("cuda", local_rank)
    else:
        dev = torch.device("cpu")
    dist = None
    if world > 1:
        import torch.distributed as dist
        if on_gpu:
            dist.init_process_group(backend, device_id=dev)
        else:
            dist.init_process_group(backend, rank=rank, world_size=world)
    B = None
    if on_gpu:
        import __graft_entry__ as entry
        if local_rank == 0:
            entry.build()
        if dist is not None:
            dist.barrier()
        from paper_2507_00715_b200 import binding as B

    if on_gpu and args.profile_kernel:
        profile_one_kernel(w, dev, args.profile_kernel)
        return

    if on_gpu and args.sweep_k:
        sweep_split_layer(w, dev, [int(x) for x in args.sweep_k.split(",")], args)
        return

    w_rank = replicas.rank_workload(w, rank)
    job = GpuJob(w_rank, dev) if on_gpu else job_factory(w_rank, dev, rank)
    peaks = read_peaks()

    def barrier():
        if dist is not None:
            dist.barrier()
        if on_gpu:
            torch.cuda.synchronize()

    n0 = B.earn_launch_count() if on_gpu else 0
    job.step()                                   # first pass: plain launches (also sets per-kernel attributes)
    launches_per_step = (B.earn_launch_count() - n0) if on_gpu else getattr(job, "launches_per_step", 0)
    if on_gpu:
        torch.cuda.synchronize()
        if not args.no_graphs:
            job.capture_graphs()                 # the same launches, recorded once, replayed per step
    for _ in range(args.warmup):
        job.step()
    barrier()
    sampler = ClockSampler(local_rank) if rank == 0 and on_gpu else None
    timer = DeviceTimer() if on_gpu else HostTimer()
    timer.start()
    for _ in range(args.steps):
        job.step(record=True)
    timer.stop()
    barrier()
    launches = launches_per_step * args.steps
    clocks = sampler.stop() if sampler else None
    elapsed = replicas.max_over_ranks(timer.seconds(), dist, dev)
    ranks_ran = replicas.count_ranks(dist, dev)
    assert job.device_status() == 0, "a device-side wait timed out"
    t_step = elapsed / args.steps
    value = replicas.job_throughput(tokens_per_step, ranks_ran, t_step)

    # rooflines from the events recorded at the segment boundaries INSIDE the timed region
    alg = algorithmic(w)
    alg["register_layer"] = dict(flops=alg["compact"]["flops"] + alg["register"]["flops"],
                                 bytes=alg["compact"]["bytes"] + alg["register"]["bytes"])
    # decode segments cover all T steps: quote the average step's cache length
    s_mid = (w.decode_steps + 1) / 2.0
    es, Bq = (4 if w.dtype == "f32" else 2), w.batch * w.beams
    qo = 2 * Bq * w.n_q_heads * w.head_dim * es + 4 * Bq * w.n_kv_heads * w.head_dim * es
    alg["decode_compact"]["bytes"] = 2 * w.batch * (w.n_regs + w.beams * s_mid) * w.n_kv_heads * w.head_dim * es + qo
    alg["decode_full"]["bytes"] = 2 * (int(lens.sum()) + Bq * s_mid) * w.n_kv_heads * w.head_dim * es + qo
    traffic = read_traffic(w.name)
    rooflines = {}
    for kind, (sec, per_step, share) in job.segment_times().items():
        a = alg[kind]
        r = {"kernel": kind}
        if kind == "prefill":
            # tensor-bound: the burst cuBLAS figure is the stricter denominator and the one `frac` uses; the
            # sustained one (a seconds-long GEMM loop under the power cap) is printed beside it
            ach = a["flops"] / sec / 1e12
            r.update(bound="tensor", achieved=ach, peak=peaks["tflops_burst"], unit="TFLOP/s",
                     frac=ach / peaks["tflops_burst"], frac_burst=ach / peaks["tflops_burst"],
                     frac_sustained=ach / peaks["tflops_sustained"], peak_sustained=peaks["tflops_sustained"],
                     frac_nominal=ach / NOMINAL["tflops"], peak_source=peaks["source"] + " (burst bf16 GEMM)")
        else:
            ach = a["bytes"] / sec / 1e9
            r.update(bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s", frac=ach / peaks["hbm_gbs"],
                     frac_nominal=ach / NOMINAL["hbm_gbs"], peak_source=peaks["source"] + " (copy)")
        tr = traffic.get(kind)
        r.update(traffic=tr, avg_launch_ms=sec * 1e3, launches_per_step=per_step, share_of_step=share,
                 algorithmic_flops_per_launch=a["flops"], algorithmic_bytes_per_launch=a["bytes"])
        rooflines[kind] = r
    roofline = max(rooflines.values(), key=lambda r: r["share_of_step"]) if rooflines else None

    parts = None
    if on_gpu and not args.no_parts and rank == 0:
        tp = job.time_parts()
        parts = {}
        for name, sec in tp.items():
            a = alg[name]
            parts[name] = {"ms_per_launch": sec * 1e3, "GB_s": a["bytes"] / sec / 1e9, "hbm_frac": a["bytes"] / sec / 1e9 / peaks["hbm_gbs"],
                           "TFLOP_s": a["flops"] / sec / 1e12, "tensor_frac": a["flops"] / sec / 1e12 / peaks["tflops_burst"],
                           "traffic": traffic.get(name)}

    e2e = None
    if on_gpu and not args.no_e2e:
        h2d, d2h = job.setup_e2e()
        job.step_e2e()
        barrier()
        n_e2e = max(1, min(args.steps, 2))
        t2 = DeviceTimer()
        t2.start()
        for _ in range(n_e2e):
            job.step_e2e()
        t2.stop()
        barrier()
        te = replicas.max_over_ranks(t2.seconds() / n_e2e, dist, dev)
        e2e = {"value": ranks_ran * tokens_per_step / te, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "ms_per_step": te * 1e3, "steps": n_e2e}

    cpu = None
    if on_gpu and rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample = OracleSample(w, job)
        tc, cores, busy, avail = timed_oracle(sample)
        cpu = {"value": sample.tokens / tc, "unit": UNIT, "cores": cores, "kind": "oracle (numpy float64)",
               "sample": sample.desc, "seconds": tc, "cores_busy_mean": busy, "blas_threads_available": avail}

    if rank == 0:
        T, N, k = w.decode_steps, w.n_layers, w.split_k
        extra = {}
        if parts:
            t_prefill = k * parts.get("prefill", {}).get("ms_per_launch", 0) + (N - k) * (
                parts.get("compact", {}).get("ms_per_launch", 0) + parts.get("register", {}).get("ms_per_launch", 0))
            extra["prefill_tokens_per_s_isolated"] = int(lens.sum()) / (t_prefill * 1e-3) if t_prefill else None
        seg = {kind: r["avg_launch_ms"] * r["launches_per_step"] for kind, r in rooflines.items()}
        t_pre = seg.get("prefill", 0.0) + seg.get("register_layer", 0.0)
        t_dec = seg.get("decode_full", 0.0) + seg.get("decode_compact", 0.0)
        if t_pre > 0:
            extra["prefill_tokens_per_s"] = ranks_ran * int(lens.sum()) / (t_pre * 1e-3)
        if t_dec > 0:
            extra["decode_tokens_per_s"] = ranks_ran * w.batch * w.beams * T / (t_dec * 1e-3)
        earn_e, van_e = job.kv_entries(T), N * (int(lens.sum()) + w.batch * w.beams * T)
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": ranks_ran, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": t_step * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": w.dtype, "data": "synthetic", "config": config, "clocks": clocks, "e2e": e2e,
            "gpu_launches": int(launches), "roofline": roofline, "rooflines": rooflines, "cpu_baseline": cpu,
            "launch_mode": "plain" if args.no_graphs or not on_gpu else "cuda-graph replay, one graph per segment",
            "sequences_per_s": ranks_ran * w.batch / t_step, "kernels": parts, "kv_reduction": 1.0 - earn_e / van_e,
            "peaks": peaks, **extra}), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
