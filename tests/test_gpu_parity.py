"""Element-by-element parity of the CUDA library (through the C ABI) against the fp64 oracle."""
import numpy as np
import pytest
import torch

from paper_2507_00715_b200 import workloads as wl
from parity_util import run_workload_and_compare

pytestmark = pytest.mark.gpu

BASE = wl.Workload("t", batch=3, n_layers=3, split_k=1, n_q_heads=8, n_kv_heads=2, head_dim=128, dtype="bf16",
                   prompt_len=0, lens=(200, 77, 333), r_head=5, r_tail=3, decode_steps=3, beams=1, seed=11)


def test_tiny_config_fp32():
    run_workload_and_compare(wl.CONFIGS["tiny"])


def test_bf16_ragged_gqa():
    run_workload_and_compare(BASE)


def test_bf16_scattered_pages():
    run_workload_and_compare(BASE.replace(seed=12, r_head=16, r_tail=16), paged_shuffle_seed=5)


def test_bf16_beams_group6():
    run_workload_and_compare(BASE.replace(seed=13, n_q_heads=12, n_kv_heads=2, lens=(130, 64), batch=2, beams=3,
                                          decode_steps=5, r_head=8, r_tail=8))


def test_f32_head_dim_128_and_bf16_head_dim_64():
    run_workload_and_compare(BASE.replace(seed=14, dtype="f32", lens=(65, 140), batch=2, n_q_heads=4))
    run_workload_and_compare(BASE.replace(seed=15, head_dim=64, lens=(129, 70), batch=2))


@pytest.mark.parametrize("rh,rt", [(0, 4), (4, 0), (0, 0), (1, 1)])
def test_one_sided_and_no_registers(rh, rt):
    run_workload_and_compare(BASE.replace(seed=16, r_head=rh, r_tail=rt, lens=(70, 40), batch=2))


def test_registers_cover_whole_sequence_and_one_extra():
    # R == L_b for the first sequence (compaction is the identity), L_b == R + 1 for the second
    run_workload_and_compare(BASE.replace(seed=17, r_head=3, r_tail=4, lens=(7, 8, 1 + 7), batch=3))


@pytest.mark.parametrize("k", [0, 3])
def test_split_at_the_ends(k):
    # k = 0: every layer is a register layer; k = N: a vanilla model that never compacts
    run_workload_and_compare(BASE.replace(seed=18, split_k=k, lens=(90, 150), batch=2))


def test_mha_and_many_registers():
    run_workload_and_compare(BASE.replace(seed=19, n_q_heads=2, n_kv_heads=2, r_head=40, r_tail=37, lens=(100, 300), batch=2))
    # more than 128 registers: the register layers fall back to the CUDA-core kernel
    run_workload_and_compare(BASE.replace(seed=20, n_q_heads=4, n_kv_heads=2, r_head=70, r_tail=75, lens=(150, 300), batch=2))


def test_group_of_three_and_odd_register_count():
    # g*R = 3*7 = 21 rows: a ragged last row tile that straddles two heads
    run_workload_and_compare(BASE.replace(seed=21, n_q_heads=6, n_kv_heads=2, r_head=3, r_tail=4, lens=(60, 33), batch=2,
                                          beams=2, decode_steps=4))


def test_register_layers_ignore_prompt_tokens_on_the_gpu():
    """Overwriting every non-register K/V/Q row of a register layer changes nothing, bit for bit: compact cache,
    register attention and every decode output of that layer (the layer never reads those rows)."""
    from parity_util import make_session
    from oracle import earn_oracle as orc

    w = BASE.replace(seed=22, lens=(300, 129, 64), r_head=6, r_tail=5, decode_steps=3, beams=2, n_layers=2, split_k=1)
    idx = orc.register_indices(wl.seqlens(w), w.r_head, w.r_tail)
    cu = wl.cu_seqlens(w)
    keep = torch.zeros(int(cu[-1]), dtype=torch.bool)
    for b in range(w.batch):
        keep[cu[b] + torch.from_numpy(idx[b]).long()] = True
    outs = []
    for noise_seed in (None, 1234):
        ses = make_session(w)
        q, k, v = wl.layer_qkv(w, 1, "cuda")
        if noise_seed is not None:
            g = torch.Generator(device="cuda").manual_seed(noise_seed)
            for t in (q, k, v):
                noise = torch.randn(t.shape, generator=g, device="cuda").to(t.dtype)
                t[~keep.cuda()] = noise[~keep.cuda()]
        got = [ses.prefill_layer(1, q, k, v).clone(), ses.k_shared[1].clone(), ses.v_shared[1].clone()]
        for step in range(1, w.decode_steps + 1):
            parents = wl.beam_parents(w, step) if step > 1 else None
            ses.begin_step(step, None if parents is None else torch.from_numpy(parents).cuda())
            got.append(ses.decode_layer(1, step, *wl.decode_qkv(w, 1, step, "cuda")).clone())
        outs.append(got)
    for a, b in zip(*outs):
        assert torch.equal(a, b)


def test_batch_order_does_not_matter():
    """Sequences are independent (varlen packing, no padding): reversing the batch reverses the outputs."""
    from parity_util import make_session

    w = BASE.replace(seed=23, lens=(200, 77, 333), n_layers=1, split_k=1, decode_steps=0)
    cu = wl.cu_seqlens(w)
    q, k, v = wl.layer_qkv(w, 0, "cuda")
    o = make_session(w).prefill_layer(0, q, k, v)
    order = [2, 1, 0]
    pieces = lambda t: torch.cat([t[cu[b]:cu[b + 1]] for b in order])   # noqa: E731
    w2 = w.replace(lens=tuple(w.lens[b] for b in order))
    o2 = make_session(w2).prefill_layer(0, pieces(q), pieces(k), pieces(v))
    assert torch.equal(o2, pieces(o))


def test_beam_search_row_tiles_share_the_cache_pass():
    """More query rows per kv head than one 16-row tile (beams x group size > 16): two row tiles, then five row
    tiles in two groups with split-KV on a long prompt, scattered pages, and head_dim 64."""
    run_workload_and_compare(BASE.replace(seed=24, n_q_heads=8, n_kv_heads=2, lens=(150, 90), batch=2, beams=5,
                                          decode_steps=4, r_head=9, r_tail=8), paged_shuffle_seed=3)
    run_workload_and_compare(BASE.replace(seed=25, n_q_heads=8, n_kv_heads=2, lens=(1500,), batch=1, beams=20,
                                          decode_steps=3, r_head=16, r_tail=16, n_layers=2, split_k=1), check_lse=False)
    run_workload_and_compare(BASE.replace(seed=26, head_dim=64, n_q_heads=8, n_kv_heads=2, lens=(200, 64), batch=2,
                                          beams=7, decode_steps=3, r_head=4, r_tail=4))


def test_two_row_tiles_over_a_short_list():
    """Beams x group size between 17 and 32 over a compact cache of a few dozen positions (the paper's own multi-head
    setting: 20 beams, one register per side, four-token identifiers).  20 and 32 beams of a multi-head model (6 and 8
    key tiles at the last step), 18 rows left ragged by a group of 3 (the second tile mostly empty), and lists of at
    most four tiles behind a shuffled page table."""
    lens = tuple(20 + (i * 11) % 60 for i in range(6))
    run_workload_and_compare(BASE.replace(seed=41, n_q_heads=8, n_kv_heads=8, lens=lens, batch=6, beams=20,
                                          decode_steps=4, r_head=1, r_tail=1, n_layers=2, split_k=1), check_lse=False)
    run_workload_and_compare(BASE.replace(seed=42, n_q_heads=4, n_kv_heads=4, lens=lens[:3], batch=3, beams=32,
                                          decode_steps=3, r_head=2, r_tail=2, n_layers=2, split_k=1), check_lse=False)
    run_workload_and_compare(BASE.replace(seed=43, n_q_heads=6, n_kv_heads=2, lens=lens[:3], batch=3, beams=6,
                                          decode_steps=5, r_head=3, r_tail=2, n_layers=2, split_k=1), check_lse=False)
    run_workload_and_compare(BASE.replace(seed=44, n_q_heads=4, n_kv_heads=2, lens=lens[:2], batch=2, beams=9,
                                          decode_steps=2, r_head=4, r_tail=4, n_layers=2, split_k=1), paged_shuffle_seed=5,
                             check_lse=False)


def test_two_row_tiles_on_a_grid_of_many_ctas_head_dim_64():
    """20 beams of a multi-head model (two row tiles per kv head) over more (sequence, kv head) pairs than four CTAs
    per SM hold: the launch takes the shallower ring with six CTAs per SM; head_dim 64; six decode steps, so the
    private tiles outnumber a warp's ring slice; one register per side like the paper's own setting."""
    lens = tuple(12 + (i * 7) % 30 for i in range(20))
    run_workload_and_compare(BASE.replace(seed=27, head_dim=64, n_q_heads=32, n_kv_heads=32, lens=lens, batch=20, beams=20,
                                          decode_steps=6, r_head=1, r_tail=1, n_layers=2, split_k=1), check_lse=False)


def test_long_uneven_prompts_are_decoded_longest_first():
    """Prompt-cache decode of a batch whose prompts are long and uneven hands its CTAs out by decreasing length (the
    grid index is a rank; a small launch ahead of the kernel writes the rank -> sequence table): equal lengths in the
    batch exercise the tie rule; one beam (one row tile) and five beams (several row tiles)."""
    w = BASE.replace(seed=28, lens=(1200, 90, 400, 1200, 33, 1024), batch=6, n_layers=2, split_k=1, decode_steps=2)
    run_workload_and_compare(w, check_lse=False)
    run_workload_and_compare(w.replace(seed=29, beams=5), check_lse=False)


def test_long_prompt_among_empty_ones():
    """One long prompt and many empty ones (no registers): decode over an empty prompt cache sees the generated tokens
    only, and the batch is too sparse for the longest-first table to fit the plan area, so the plain order is used."""
    w = BASE.replace(seed=30, lens=(1100,) + (0,) * 69, batch=70, n_layers=1, split_k=1, r_head=0, r_tail=0, decode_steps=2)
    run_workload_and_compare(w, check_lse=False)


def test_a_wait_that_runs_out_is_reported_and_the_context_survives():
    """Failure detection without a fault: a bounded device-side wait on a barrier nothing completes gives up after
    its limit, the kernel returns normally with EARN_ERR_TIMEOUT in the status word, and the library keeps working."""
    from paper_2507_00715_b200 import binding as B
    from parity_util import make_session

    w = BASE.replace(seed=27, lens=(200, 140), batch=2, n_layers=1, split_k=1, decode_steps=0)
    ses = make_session(w)
    assert ses.device_status() == B.EARN_OK
    B.earn_selftest_wait_timeout(ses.workspace, 2_000_000)          # about a millisecond
    assert ses.device_status() == B.EARN_ERR_TIMEOUT
    B.earn_workspace_init(ses.workspace)
    assert ses.device_status() == B.EARN_OK
    run_workload_and_compare(w)                                      # the context is still usable
    with pytest.raises(B.EarnError):
        B.earn_selftest_wait_timeout(ses.workspace, 10**12)          # limit beyond a second: refused on the host


def test_prefill_logits_that_keep_rising_take_the_rescale_path():
    """Logits that grow along the sequence by far more than the lazy-rescale bound: every key tile after the first
    must raise the softmax reference, rescale the running output and redo its pass."""
    from oracle import earn_oracle as orc
    from parity_util import assert_close, make_session, to_np

    w = BASE.replace(seed=28, lens=(700, 390), batch=2, n_layers=1, split_k=1, decode_steps=0, n_q_heads=4, n_kv_heads=2)
    cu = wl.cu_seqlens(w)
    q, k, v = wl.layer_qkv(w.replace(sink_q_bias=False), 0, "cuda")
    u = torch.nn.functional.normalize(torch.randn(w.head_dim, device="cuda"), dim=0)
    pos = torch.cat([torch.arange(int(n), device="cuda") for n in wl.seqlens(w)]).float()
    # scaled logit of key j grows by about 0.35 per position: +45 per 128-key tile, +65 in the log2 domain
    k = (k.float() * 0.1 + (pos[:, None, None] * 0.35) * u).to(torch.bfloat16)
    q = (q.float() * 0.1 + (w.head_dim ** 0.5) * u).to(torch.bfloat16)
    o = make_session(w).prefill_layer(0, q, k, v)
    ref, _ = orc.causal_attention(to_np(q), to_np(k), to_np(v), cu)
    assert_close(o, ref, "bf16", "prefill with rising logits")


def test_one_token_sequences_among_long_ones():
    """Sequences of one and two tokens packed between long ones: the plan of the tensor-core prefill gets entries
    of a single valid row, compaction keeps the only token, decode sees a one-key prompt cache."""
    run_workload_and_compare(BASE.replace(seed=29, lens=(1, 300, 2, 129, 1), batch=5, r_head=1, r_tail=0, beams=2,
                                          decode_steps=2))


@pytest.mark.parametrize("shape", ["one_row_tile", "several_row_tiles", "fp32", "short_list_head_dim_64"])
def test_private_segment_behind_a_page_table(shape):
    """The generated tokens live in scattered 16-token pages (one table for every layer) instead of flat slabs: 18
    decode steps cross a page boundary, beams are re-parented every step, every decode kernel family takes a turn."""
    kw = {"one_row_tile": dict(n_q_heads=4, n_kv_heads=2, beams=3),                 # streaming + short-list kernels
          "several_row_tiles": dict(n_q_heads=8, n_kv_heads=2, beams=5),             # 20 query rows per kv head
          "fp32": dict(dtype="f32", n_q_heads=4, n_kv_heads=2, beams=2, head_dim=64),
          "short_list_head_dim_64": dict(head_dim=64, n_q_heads=4, n_kv_heads=2, beams=2)}[shape]
    w = BASE.replace(seed=23, lens=(90, 40), batch=2, n_layers=2, split_k=1, r_head=4, r_tail=4, decode_steps=18, **kw)
    run_workload_and_compare(w, check_lse=False, paged_private_seed=9, paged_shuffle_seed=3)


@pytest.mark.parametrize("kw", [dict(), dict(r_head=16, r_tail=16, paged=True), dict(n_q_heads=6, n_kv_heads=2, r_head=3, r_tail=4),
                                dict(r_head=0, r_tail=4), dict(r_head=40, r_tail=37, n_q_heads=2, n_kv_heads=2, lens=(100, 300), batch=2),
                                dict(r_head=3, r_tail=4, lens=(7, 8, 300)), dict(head_dim=64)])
def test_compaction_and_register_attention_in_one_launch(kw):
    """earn_compact_register_attn leaves the cache pages and the index list bit-identical to earn_compact_kv's and returns
    earn_register_attn's output (here: bit-identical too, the arithmetic is the same kernel's), and both match the oracle."""
    from parity_util import assert_close, make_session, to_np
    from oracle import earn_oracle as orc
    kw = dict(kw)
    paged = kw.pop("paged", False)
    w = BASE.replace(seed=24, n_layers=2, split_k=1, decode_steps=0, **kw)
    cu = wl.cu_seqlens(w)
    idx = orc.register_indices(wl.seqlens(w), w.r_head, w.r_tail)
    q, k, v = wl.layer_qkv(w, 1, "cuda")
    two = make_session(w, paged_shuffle_seed=5 if paged else None)
    o_two = two.prefill_layer(1, q, k, v)
    one = make_session(w, paged_shuffle_seed=5 if paged else None)
    o_one = one.register_layer_fused(1, q, k, v)
    torch.cuda.synchronize()
    assert torch.equal(one.k_shared[1], two.k_shared[1]) and torch.equal(one.v_shared[1], two.v_shared[1])
    assert torch.equal(one.reg_idx, two.reg_idx)
    assert torch.equal(o_one, o_two)
    qn, kn, vn = to_np(q), to_np(k), to_np(v)
    assert_close(o_one, orc.register_attention(orc.compact(qn, cu, idx), orc.compact(kn, cu, idx), orc.compact(vn, cu, idx)),
                 w.dtype, "fused register layer")
    assert np.array_equal(one.reg_idx.cpu().numpy()[:, :w.n_regs], idx)
