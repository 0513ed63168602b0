"""Runs a workload through the CUDA library and through the oracle and compares every output."""
import numpy as np
import torch

from oracle import earn_oracle as orc
from paper_2507_00715_b200 import workloads as wl
from paper_2507_00715_b200.session import EarnSession

# bf16 inputs with fp32 accumulation, and the fp32 debug path
TOL = {"bf16": dict(max_abs=2e-2, mean_abs=2e-3), "f32": dict(max_abs=1e-5, mean_abs=1e-6)}


def to_np(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a (bf16 or fp32) tensor to a float32 numpy array on the host."""
    return t.detach().float().cpu().numpy()


def assert_close(got: torch.Tensor, ref: np.ndarray, dtype: str, what: str):
    g = got.detach().double().cpu().numpy()
    assert g.shape == ref.shape, (what, g.shape, ref.shape)
    if g.size == 0:
        return
    assert np.isfinite(g).all(), f"{what}: non-finite output"
    err = np.abs(g - ref)
    t = TOL[dtype]
    assert err.max() <= t["max_abs"], f"{what}: max abs err {err.max():.3e} > {t['max_abs']}"
    assert err.mean() <= t["mean_abs"], f"{what}: mean abs err {err.mean():.3e} > {t['mean_abs']}"


def make_session(w: wl.Workload, **kw) -> EarnSession:
    return EarnSession(w.n_layers, w.split_k, w.n_q_heads, w.n_kv_heads, w.head_dim, w.torch_dtype,
                       wl.cu_seqlens(w), w.r_head, w.r_tail, beams=w.beams, max_new=max(w.decode_steps, 1),
                       device="cuda", **kw)


def run_workload_and_compare(w: wl.Workload, check_lse=True, **session_kw):
    """Whole hot path, every element compared (use on sizes the oracle finishes in seconds)."""
    cu = wl.cu_seqlens(w)
    lens = wl.seqlens(w)
    idx = orc.register_indices(lens, w.r_head, w.r_tail)
    ses = make_session(w, **session_kw)
    states = []
    for layer in range(w.n_layers):
        q, k, v = wl.layer_qkv(w, layer, "cuda")
        qn, kn, vn = to_np(q), to_np(k), to_np(v)
        if layer < w.split_k:
            lse = torch.empty(w.n_q_heads, int(cu[-1]), device="cuda", dtype=torch.float32) if check_lse else None
            o = ses.prefill_layer(layer, q, k, v, lse=lse)
            ref, ref_lse = orc.causal_attention(qn, kn, vn, cu)
            assert_close(o, ref, w.dtype, f"prefill layer {layer}")
            if check_lse and int(cu[-1]) > 0:
                d = np.abs(lse.double().cpu().numpy() - ref_lse).max()
                assert d <= (1e-4 if w.dtype == "f32" else 2e-2), f"lse layer {layer}: {d}"
            shared_k = [kn[cu[b]:cu[b + 1]] for b in range(w.batch)]
            shared_v = [vn[cu[b]:cu[b + 1]] for b in range(w.batch)]
        else:
            o = ses.prefill_layer(layer, q, k, v)
            kc, vc, qc = orc.compact(kn, cu, idx), orc.compact(vn, cu, idx), orc.compact(qn, cu, idx)
            # bit-exact: indices and cache contents (through the page table)
            R = w.n_regs
            if R > 0:
                assert np.array_equal(ses.reg_idx.cpu().numpy()[:, :R], idx)
                pages = (ses.block_table.cpu().numpy() if ses.block_table is not None else
                         np.arange(ses.n_pages).reshape(w.batch, ses.pages_per_seq))
                ks = to_np(ses.k_shared[layer])
                vs = to_np(ses.v_shared[layer])
                for b in range(w.batch):
                    for m in range(R):
                        pg = pages[b, m // 16]
                        assert ks[pg, m % 16].tobytes() == kc[b, m].tobytes(), ("k compact", layer, b, m)
                        assert vs[pg, m % 16].tobytes() == vc[b, m].tobytes(), ("v compact", layer, b, m)
                assert to_np(ses.last_q_reg).tobytes() == qc.tobytes()
            assert_close(o, orc.register_attention(qc, kc, vc), w.dtype, f"register layer {layer}")
            shared_k = [kc[b] for b in range(w.batch)]
            shared_v = [vc[b] for b in range(w.batch)]
        states.append(orc.DecodeState(shared_k, shared_v, w.beams))
    for step in range(1, w.decode_steps + 1):
        parents = wl.beam_parents(w, step) if w.beams > 1 and step > 1 else None
        ses.begin_step(step, None if parents is None else torch.from_numpy(parents).cuda())
        for layer in range(w.n_layers):
            q, k, v = wl.decode_qkv(w, layer, step, "cuda")
            o = ses.decode_layer(layer, step, q, k, v)
            ref = states[layer].step(to_np(q), to_np(k), to_np(v), parents)
            assert_close(o, ref, w.dtype, f"decode step {step} layer {layer}")
    assert ses.device_status() == 0
    return ses
