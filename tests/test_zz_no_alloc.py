"""The decode entry point that allocates nothing (earn_decode_attn_static) against the ordinary one and the oracle.

Collected last on purpose: a run that stops at the first failure has then already been through every other test.
The caller this entry point exists for cannot allocate device memory (its host owns the memory pool, or it
cannot afford cudaMalloc's synchronisation), so the library brings a fixed scratch array of its own.  The test
passes the same inputs to both entry points, through the C ABI, and expects the same outputs, twice in a row,
because the scratch array is shared by all calls and keeps what the previous call left in it.  The static call's
output is also held against the CPU oracle's decode step, so the test stands without the ordinary entry point,
and the device allocator's state is read before and after the static calls: it must not move.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import earn_oracle as orc
from paper_2507_00715_b200 import binding as B
from paper_2507_00715_b200 import workloads as wl
from parity_util import TOL, make_session, to_np

SHAPES = {
    # one long sequence and two kv heads: too few CTAs to fill the GPU unsplit, so the prompt-cache layer runs
    # split-KV and the scratch memory (tickets + partials) is really used; one row tile
    "split_one_row_tile": dict(batch=1, n_q_heads=8, n_kv_heads=2, lens=(2048,), beams=2),
    # ten beams x group of 4 = 40 query rows per kv head: the several-row-tile kernel, split over the prompt
    "split_several_row_tiles": dict(batch=1, n_q_heads=8, n_kv_heads=2, lens=(1536,), beams=10),
    # two long prompts more than 1.25x apart: the longest-first order table is written into the scratch's plan area
    "ragged_order_table": dict(batch=2, n_q_heads=8, n_kv_heads=2, lens=(1100, 2300), beams=1),
}


@pytest.mark.gpu
@pytest.mark.parametrize("shape", sorted(SHAPES))
@pytest.mark.parametrize("early_layer", [True, False])
def test_static_scratch_decode_matches_workspace_decode_and_oracle(early_layer, shape):
    w = wl.Workload("noalloc", n_layers=2, split_k=1, head_dim=128, dtype="bf16", prompt_len=0, r_head=16, r_tail=16,
                    decode_steps=2, seed=31, **SHAPES[shape])
    ses = make_session(w)
    assert B.earn_workspace_bytes(ses.model, ses.batch, w.beams) <= B.STATIC_SCRATCH_BYTES
    cu = wl.cu_seqlens(w)
    idx = orc.register_indices(wl.seqlens(w), w.r_head, w.r_tail)
    layer = 0 if early_layer else 1
    for l in range(w.n_layers):
        q, k, v = wl.layer_qkv(w, l, "cuda")
        ses.prefill_layer(l, q, k, v)
        if l == layer:
            kn, vn = to_np(k), to_np(v)
            if early_layer:
                shared = [kn[cu[b]:cu[b + 1]] for b in range(w.batch)], [vn[cu[b]:cu[b + 1]] for b in range(w.batch)]
            else:
                shared = list(orc.compact(kn, cu, idx)), list(orc.compact(vn, cu, idx))
    state = orc.DecodeState(shared[0], shared[1], w.beams)
    tol = TOL[w.dtype]
    # everything the loop needs is allocated before the allocator's state is read
    steps = []
    for step in (1, 2):
        q, k_new, v_new = wl.decode_qkv(w, layer, step, "cuda")
        parents = wl.beam_parents(w, step) if w.beams > 1 and step > 1 else None
        steps.append((step, q, k_new, v_new, parents, None if parents is None else torch.from_numpy(parents).cuda(),
                      torch.empty_like(q), torch.full_like(q, float("nan"))))
    # The set-up call: the first use of the entry point on a device looks up the scratch array's address, and the
    # driver, which loads a module's code and data on first use, only now takes the array's 8 MiB (and the kernels'
    # code) from device memory.  It is step 1 itself, which the loop below repeats with the same result.
    step, q, k_new, v_new, _, _, ref, got = steps[0]
    B.earn_decode_attn(ses.model, ses.batch, layer, step, q, k_new, v_new, ses.cache(layer), ref,
                       ses.k_full[layer], ses.v_full[layer], ses.workspace)
    B.earn_decode_attn_static(ses.model, ses.batch, layer, step, q, k_new, v_new, ses.cache(layer), got,
                              ses.k_full[layer], ses.v_full[layer])
    if steps[1][5] is not None:   # the re-parenting kernel of step 2 is loaded too (into a table the loop rewrites)
        B.earn_beam_reparent(w.batch, w.beams, ses.max_new, 2, steps[1][5], None, ses.lineage[1])
    got.fill_(float("nan"))
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0 = torch.cuda.memory_allocated()
    for step, q, k_new, v_new, parents, parents_dev, ref, got in steps:   # two calls in a row share the scratch array
        ses.begin_step(step, parents_dev)
        B.earn_decode_attn(ses.model, ses.batch, layer, step, q, k_new, v_new, ses.cache(layer), ref,
                           ses.k_full[layer], ses.v_full[layer], ses.workspace)
        B.earn_decode_attn_static(ses.model, ses.batch, layer, step, q, k_new, v_new, ses.cache(layer), got,
                                  ses.k_full[layer], ses.v_full[layer])
        torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == alloc0, "a tensor was allocated during the static calls"
    assert torch.cuda.mem_get_info()[0] == free0, "device memory was taken or returned during the static calls"
    for step, q, k_new, v_new, parents, parents_dev, ref, got in steps:
        assert torch.isfinite(got.float()).all()
        err = (got.double() - ref.double()).abs()
        assert err.max().item() <= tol["max_abs"] and err.mean().item() <= tol["mean_abs"], (step, err.max().item())
        want = state.step(to_np(q), to_np(k_new), to_np(v_new), parents)
        err = np.abs(got.double().cpu().numpy() - want)
        assert err.max() <= tol["max_abs"] and err.mean() <= tol["mean_abs"], ("oracle", step, err.max(), err.mean())
    assert ses.device_status() == 0


def test_static_scratch_rejects_a_batch_that_needs_more_than_it_holds():
    # host-side check only: nothing is launched, no device is touched
    import __graft_entry__ as entry
    entry.build()
    lib = B.lib()
    lens = np.full(128, 2048, dtype=np.int32)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    batch = B.EarnBatch(128, int(cu[-1]), 2048, 0x1000, cu.ctypes.data, 16, 16)
    model = B.make_model(32, 8, 32, 8, 128, "bf16")
    assert lib.earn_workspace_bytes(C.byref(model), C.byref(batch), 10) > B.STATIC_SCRATCH_BYTES
    cache = B.make_cache(0x1000, 0x1000, None, 2, 256, 0x1000, 0x1000, None, 10, 4, None)
    rc = lib.earn_decode_attn_static(C.byref(model), C.byref(batch), 8, 1, 0x1000, 0x1000, 0x1000, None, None,
                                     C.byref(cache), 0x1000, None)
    assert rc == B.EARN_ERR_WORKSPACE
    assert lib.earn_status_string(rc).decode().startswith("workspace")
