"""Beam selection (earn_beam_topk) against the oracle: parents, tokens and scores bit for bit, and a decode step driven by
the selected parents (selection -> re-parenting -> decode, with no host round trip in between)."""
import numpy as np
import pytest
import torch

from oracle import earn_oracle as orc
from paper_2507_00715_b200 import binding as B
from paper_2507_00715_b200 import workloads as wl
from parity_util import assert_close, make_session, to_np

pytestmark = pytest.mark.gpu


def run_topk(logprobs: torch.Tensor, scores, beams: int, n_live: int):
    rows, vocab = logprobs.shape
    batch = rows // beams
    ws = torch.empty(B.earn_beam_topk_workspace_bytes(batch, beams, vocab), dtype=torch.uint8, device="cuda")
    parent = torch.full((rows,), -7, dtype=torch.int32, device="cuda")
    token = torch.full((rows,), -7, dtype=torch.int32, device="cuda")
    new = torch.full((rows,), float("nan"), dtype=torch.float32, device="cuda")
    B.earn_beam_topk(batch, beams, n_live, vocab, logprobs, scores, parent, token, new, ws)
    torch.cuda.synchronize()
    return parent, token, new


def check(logprobs, scores, beams, n_live=None):
    n_live = beams if n_live is None else n_live
    parent, token, new = run_topk(logprobs, scores, beams, n_live)
    sc = np.zeros(logprobs.shape[0], np.float32) if scores is None else scores.cpu().numpy()
    p_ref, t_ref, s_ref = orc.beam_topk(logprobs.cpu().numpy(), sc, beams, n_live)
    assert np.array_equal(parent.cpu().numpy(), p_ref)
    assert np.array_equal(token.cpu().numpy(), t_ref)
    assert np.array_equal(new.cpu().numpy(), s_ref)          # the same fp32 sum on both sides


def _w(batch, beams, seed=41):
    return wl.Workload("beam", batch=batch, n_layers=2, split_k=1, n_q_heads=4, n_kv_heads=2, head_dim=128, dtype="bf16",
                       prompt_len=64, r_head=2, r_tail=2, decode_steps=3, beams=beams, seed=seed)


@pytest.mark.parametrize("batch,beams,vocab", [(3, 4, 11), (2, 20, 1000), (5, 20, 32000), (2, 32, 8191), (7, 1, 5000),
                                               (2, 20, 152064)])
def test_topk_random_logprobs(batch, beams, vocab):
    """One chunk, a few chunks with a ragged last one, the vocabularies of the paper's two backbones (32K and 152K
    tokens: 79 and 372 chunks per sequence), the widest beam, greedy decoding."""
    w = _w(batch, beams)
    lp = wl.beam_logprobs(w, 2, vocab, "cuda")
    g = torch.Generator(device="cuda")
    g.manual_seed(5)
    scores = -3.0 * torch.rand(batch * beams, generator=g, device="cuda")
    check(lp, scores, beams)
    check(lp, None, beams, n_live=1)                         # first step: only beam 0 of every sequence offers candidates


def test_topk_with_most_of_the_vocabulary_forbidden():
    """Identifier generation restricted to valid tokens: 30 finite log-probabilities per row among 32000, fewer finite
    candidates in most chunks than beams, and in one case fewer in the whole sequence than beams (ties among -inf)."""
    w = _w(3, 20)
    check(wl.beam_logprobs(w, 1, 32000, "cuda", allowed=30), None, 20)
    lp = wl.beam_logprobs(w, 1, 32000, "cuda", allowed=30)
    check(lp, None, 20, n_live=1)                            # 30 finite candidates >= 20 beams
    lp2 = wl.beam_logprobs(_w(2, 20), 1, 9000, "cuda", allowed=1)
    check(lp2, None, 20)                                     # 20 finite candidates for 20 beams
    check(lp2, None, 20, n_live=3)                           # 3 finite candidates: the other 17 slots are ties among -inf


def test_topk_flat_and_tied_distributions():
    """Every candidate equal (the first W flat indices win, in order), and planted exact ties across beams and chunks."""
    flat = torch.zeros(2 * 8, 20000, device="cuda")
    check(flat, None, 8)
    check(flat, torch.zeros(16, device="cuda"), 8, n_live=2)
    w = _w(2, 8)
    lp = wl.beam_logprobs(w, 3, 20000, "cuda")
    top = lp.max()
    lp[0, 19999] = lp[3, 7] = lp[5, 12345] = lp[5, 12346] = top + 1.0      # four equal best candidates in sequence 0
    lp[8:, 500] = top + 2.0                                                  # eight equal best in sequence 1, one per beam
    check(lp, None, 8)
    two_valued = (torch.arange(16 * 20000, device="cuda").reshape(16, 20000) % 3 == 0).float()   # a third of all candidates tie for first
    check(two_valued, None, 8)


def test_topk_values_that_keep_rising_or_arrive_late():
    """What the running threshold of a CTA that walks several chunks must survive: scores that rise with the flat index
    (every candidate of every later chunk beats the W-th best so far), a rise that stops half way (the pre-filter then
    passes nothing), the best W hidden in the last chunk, equal values on both sides of a chunk boundary, and a batch
    large enough for every CTA to take many chunks."""
    rows, vocab, beams = 2 * 20, 40000, 20
    rising = torch.arange(rows * vocab, device="cuda", dtype=torch.float32).reshape(rows, vocab) * 1e-3
    check(rising - 100.0, None, beams)
    check(-rising, None, beams)                                   # falling: only the first chunk matters
    half = torch.minimum(rising, torch.full_like(rising, 300.0))  # rises, then a long flat top: ties by smallest index
    check(half, None, beams)
    w = _w(2, beams)
    lp = wl.beam_logprobs(w, 1, vocab, "cuda")
    lp[19, vocab - 25:] = lp.max() + 1.0 + torch.arange(25, device="cuda", dtype=torch.float32)   # the best, at the very end
    lp[39, 8192 * 3 - 2:8192 * 3 + 2] = lp.max() + 0.5            # four equal values across a chunk boundary
    check(lp, wl.beam_logprobs(w, 2, 7, "cuda")[:, 0].contiguous(), beams)
    big = _w(64, beams)
    check(wl.beam_logprobs(big, 4, 32000, "cuda"), None, beams)   # 64 x 79 chunks: a dozen chunks per CTA
    check(wl.beam_logprobs(big, 5, 32000, "cuda"), None, beams, n_live=1)   # first decode step: one live beam, four chunks


def test_selection_then_reparenting_then_decode():
    """A decode step whose parents come from the selection kernel: topk -> earn_beam_reparent -> earn_decode_attn on the
    device, against the oracle's selection feeding the oracle's decode state."""
    w = _w(3, 5)
    vocab = 777
    cu = wl.cu_seqlens(w)
    idx = orc.register_indices(wl.seqlens(w), w.r_head, w.r_tail)
    ses = make_session(w)
    states = []
    for layer in range(w.n_layers):
        q, k, v = wl.layer_qkv(w, layer, "cuda")
        ses.prefill_layer(layer, q, k, v)
        kn, vn = to_np(k), to_np(v)
        if layer < w.split_k:
            states.append(orc.DecodeState([kn[cu[b]:cu[b + 1]] for b in range(w.batch)],
                                          [vn[cu[b]:cu[b + 1]] for b in range(w.batch)], w.beams))
        else:
            states.append(orc.DecodeState(list(orc.compact(kn, cu, idx)), list(orc.compact(vn, cu, idx)), w.beams))
    rows = w.batch * w.beams
    ws = torch.empty(B.earn_beam_topk_workspace_bytes(w.batch, w.beams, vocab), dtype=torch.uint8, device="cuda")
    scores = [torch.zeros(rows, device="cuda"), torch.zeros(rows, device="cuda")]
    parent = torch.zeros(rows, dtype=torch.int32, device="cuda")
    token = torch.zeros(rows, dtype=torch.int32, device="cuda")
    ref_scores = np.zeros(rows, np.float32)
    p_ref = None
    for step in range(1, w.decode_steps + 1):
        if step >= 2:                                        # the survivors of step - 1 take over their parents' histories
            ses.begin_step(step, parent)
        for layer in range(w.n_layers):
            dq, dk, dv = wl.decode_qkv(w, layer, step, "cuda")
            o = ses.decode_layer(layer, step, dq, dk, dv)
            ref = states[layer].step(to_np(dq), to_np(dk), to_np(dv), p_ref)
            assert_close(o, ref, w.dtype, f"decode step {step} layer {layer}")
        # the model's output layer would give the next token's log-probabilities here; the selection reads them on the device
        lp = wl.beam_logprobs(w, step, vocab, "cuda")
        n_live = 1 if step == 1 else w.beams                 # after the first step every beam holds the same history
        cur, nxt = scores[step & 1], scores[(step + 1) & 1]
        B.earn_beam_topk(w.batch, w.beams, n_live, vocab, lp, cur, parent, token, nxt, ws)
        p_ref, t_ref, ref_scores = orc.beam_topk(lp.cpu().numpy(), ref_scores, w.beams, n_live)
        assert np.array_equal(parent.cpu().numpy(), p_ref) and np.array_equal(token.cpu().numpy(), t_ref)
        assert np.array_equal(nxt.cpu().numpy(), ref_scores)
    assert ses.device_status() == 0
