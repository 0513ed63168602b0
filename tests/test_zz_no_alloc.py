"""The decode entry point that allocates nothing (earn_decode_attn_static) against the ordinary one.

Collected last on purpose: a run that stops at the first failure has then already been through every other test.
The caller this entry point exists for cannot allocate device memory (its host owns the memory pool, or it
cannot afford cudaMalloc's synchronisation), so the library brings a fixed scratch array of its own.  The test
passes the same inputs to both entry points, through the C ABI, and expects the same outputs, twice in a row,
because the scratch array is shared by all calls and keeps what the previous call left in it.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2507_00715_b200 import binding as B
from paper_2507_00715_b200 import workloads as wl
from parity_util import TOL


def _session(w):
    from parity_util import make_session
    return make_session(w)


@pytest.mark.gpu
@pytest.mark.parametrize("early_layer", [True, False])
def test_static_scratch_decode_matches_workspace_decode(early_layer):
    # one long sequence and two kv heads: too few CTAs to fill the GPU unsplit, so the prompt-cache layer runs
    # split-KV and the scratch memory (tickets + partials) is really used
    w = wl.Workload("noalloc", batch=1, n_layers=2, split_k=1, n_q_heads=8, n_kv_heads=2, head_dim=128, dtype="bf16",
                    prompt_len=0, lens=(2048,), r_head=16, r_tail=16, decode_steps=2, beams=2, seed=31)
    ses = _session(w)
    assert B.earn_workspace_bytes(ses.model, ses.batch, w.beams) <= B.STATIC_SCRATCH_BYTES
    for layer in range(w.n_layers):
        ses.prefill_layer(layer, *wl.layer_qkv(w, layer, "cuda"))
    layer = 0 if early_layer else 1
    tol = TOL[w.dtype]
    for step in (1, 2):                                  # two calls in a row share the scratch array
        q, k_new, v_new = wl.decode_qkv(w, layer, step, "cuda")
        ref = torch.empty_like(q)
        B.earn_decode_attn(ses.model, ses.batch, layer, step, q, k_new, v_new, ses.cache(layer), ref,
                           ses.k_full[layer], ses.v_full[layer], ses.workspace)
        got = torch.full_like(q, float("nan"))
        B.earn_decode_attn_static(ses.model, ses.batch, layer, step, q, k_new, v_new, ses.cache(layer), got,
                                  ses.k_full[layer], ses.v_full[layer])
        torch.cuda.synchronize()
        err = (got.double() - ref.double()).abs()
        assert torch.isfinite(got.float()).all()
        assert err.max().item() <= tol["max_abs"] and err.mean().item() <= tol["mean_abs"], (step, err.max().item())
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
