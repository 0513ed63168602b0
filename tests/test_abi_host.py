"""The C-ABI library loads without a GPU, exports every symbol the header declares, and rejects bad
arguments on the host before anything is launched."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2507_00715_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    import __graft_entry__ as entry
    entry.build()
    return B.lib()


def declared_functions():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(earn_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = declared_functions()
    assert {"earn_prefill_attn", "earn_compact_kv", "earn_register_attn", "earn_decode_attn"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/ but not exported"
        assert n in B.SYMBOLS, f"{n} has no python binding"
    assert lib.earn_version() >= 100
    assert lib.earn_status_string(B.EARN_ERR_TIMEOUT).decode().startswith("device-side")


class FakeBatch:
    """earn_batch_t over host memory only; the device pointer is a dummy never dereferenced on the host."""

    def __init__(self, lens, rh, rt, max_seqlen=None, total=None):
        self.cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
        self.c = B.EarnBatch(len(lens), int(self.cu[-1]) if total is None else total,
                             int(max(lens)) if max_seqlen is None else max_seqlen, 0x1000, self.cu.ctypes.data, rh, rt)


def call_prefill(lib, model, batch, layer, q=0x1000, ws=0x1000, ws_bytes=1 << 20):
    return lib.earn_prefill_attn(C.byref(model), C.byref(batch.c), layer, q, 0x1000, 0x1000, 0x1000, None, ws,
                                 ws_bytes, None)


def test_host_validation_prefill(lib):
    m = B.make_model(4, 2, 8, 2, 128, "bf16")
    ok = FakeBatch([10, 20], 2, 2)
    assert call_prefill(lib, m, ok, 2) == B.EARN_ERR_INVALID_ARG          # layer on the register side of k
    assert call_prefill(lib, m, ok, -1) == B.EARN_ERR_INVALID_ARG
    assert call_prefill(lib, m, ok, 0, q=0) == B.EARN_ERR_INVALID_ARG       # null tensor
    assert call_prefill(lib, m, ok, 0, q=0x1008) == B.EARN_ERR_INVALID_ARG  # misaligned tensor
    assert call_prefill(lib, m, ok, 0, ws=0) == B.EARN_ERR_WORKSPACE
    assert call_prefill(lib, m, FakeBatch([10, 3], 2, 2), 0) == B.EARN_ERR_INVALID_ARG   # registers exceed a sequence
    assert call_prefill(lib, m, FakeBatch([10, 20], 2, 2, max_seqlen=15), 0) == B.EARN_ERR_INVALID_ARG
    assert call_prefill(lib, m, FakeBatch([10, 20], 2, 2, total=31), 0) == B.EARN_ERR_INVALID_ARG
    assert call_prefill(lib, B.make_model(4, 5, 8, 2, 128, "bf16"), ok, 0) == B.EARN_ERR_INVALID_ARG   # k > N
    assert call_prefill(lib, B.make_model(4, 2, 8, 3, 128, "bf16"), ok, 0) == B.EARN_ERR_INVALID_ARG   # Hq % Hkv
    assert call_prefill(lib, B.make_model(4, 2, 8, 2, 96, "bf16"), ok, 0) == B.EARN_ERR_UNSUPPORTED    # head_dim
    assert call_prefill(lib, m, FakeBatch([], 0, 0, max_seqlen=0), 0) == B.EARN_OK                       # empty batch


def test_host_validation_compact_register_decode(lib):
    m = B.make_model(4, 2, 8, 2, 128, "bf16")
    b = FakeBatch([40, 50], 10, 10)
    good = B.make_cache(0x1000, 0x1000, None, 2, 4, 0x1000, 0x1000, None, 1, 4, None)
    small = B.make_cache(0x1000, 0x1000, None, 1, 4, 0x1000, 0x1000, None, 1, 4, None)     # 20 rows need 2 pages
    few = B.make_cache(0x1000, 0x1000, None, 2, 3, 0x1000, 0x1000, None, 1, 4, None)       # identity table needs 4 pages

    def compact(layer, cache, q=None, qreg=None):
        return lib.earn_compact_kv(C.byref(m), C.byref(b.c), layer, 0x1000, 0x1000, q, qreg, C.byref(cache), None)

    assert compact(1, good) == B.EARN_ERR_INVALID_ARG             # a full layer is never compacted
    assert compact(4, good) == B.EARN_ERR_INVALID_ARG
    assert compact(2, small) == B.EARN_ERR_INVALID_ARG
    assert compact(2, few) == B.EARN_ERR_INVALID_ARG
    assert compact(2, good, q=0x1000, qreg=None) == B.EARN_ERR_INVALID_ARG   # q without a destination

    def reg(layer, ws=0x1000):
        return lib.earn_register_attn(C.byref(m), C.byref(b.c), layer, 0x1000, C.byref(good), 0x1000, ws, 1 << 20, None)

    assert reg(0) == B.EARN_ERR_INVALID_ARG
    assert reg(2, ws=0) == B.EARN_ERR_WORKSPACE

    def dec(layer, step, cache=good, kfull=None, ws_bytes=1 << 30):
        return lib.earn_decode_attn(C.byref(m), C.byref(b.c), layer, step, 0x1000, 0x1000, 0x1000, kfull, kfull,
                                    C.byref(cache), 0x1000, 0x1000, ws_bytes, None)

    assert dec(0, 1) == B.EARN_ERR_INVALID_ARG                    # a full layer needs the prompt K/V
    assert dec(2, 0) == B.EARN_ERR_INVALID_ARG                    # steps are 1-based
    assert dec(2, 5) == B.EARN_ERR_INVALID_ARG                    # beyond max_new
    assert dec(2, 1, ws_bytes=256) == B.EARN_ERR_WORKSPACE
    assert dec(4, 1) == B.EARN_ERR_INVALID_ARG
    # a paged private segment: 20 generated tokens need two pages per beam
    paged = B.make_cache(0x1000, 0x1000, None, 2, 4, 0x1000, 0x1000, None, 1, 20, None, 0x7000, 1, 8)
    assert dec(2, 1, cache=paged) == B.EARN_ERR_INVALID_ARG
    assert dec(2, 1, cache=B.make_cache(0x1000, 0x1000, None, 2, 4, 0x1000, 0x1000, None, 1, 20, None, 0x7000, 2, 0)) == B.EARN_ERR_INVALID_ARG

    assert lib.earn_beam_reparent(2, 3, 4, 2, 0x1000, 0x2000, 0x2000, None) == B.EARN_ERR_INVALID_ARG   # aliasing tables
    assert lib.earn_beam_reparent(2, 3, 4, 5, 0x1000, None, 0x2000, None) == B.EARN_ERR_INVALID_ARG


def test_host_validation_decode_static(lib):
    """The entry point with the built-in scratch runs the ordinary decode call's checks before it sizes or clears
    anything: a malformed model must come back as an error code, not as a crash of the host process."""
    b = FakeBatch([40, 50], 10, 10)
    good = B.make_cache(0x1000, 0x1000, None, 2, 4, 0x1000, 0x1000, None, 1, 4, None)

    def dec(model, layer=2, step=1, cache=good, q=0x1000, batch=b):
        return lib.earn_decode_attn_static(C.byref(model), C.byref(batch.c), layer, step, q, 0x1000, 0x1000, None, None,
                                           C.byref(cache), 0x1000, None)

    n0 = lib.earn_launch_count()
    m = B.make_model(4, 2, 8, 2, 128, "bf16")
    assert dec(B.make_model(4, 2, 8, 0, 128, "bf16")) == B.EARN_ERR_INVALID_ARG     # no kv heads: no division by zero
    assert dec(B.make_model(4, 2, 8, 3, 128, "bf16")) == B.EARN_ERR_INVALID_ARG     # Hq % Hkv
    assert dec(B.make_model(4, 2, 8, 2, 96, "bf16")) == B.EARN_ERR_UNSUPPORTED
    assert dec(m, step=0) == B.EARN_ERR_INVALID_ARG
    assert dec(m, step=5) == B.EARN_ERR_INVALID_ARG
    assert dec(m, layer=4) == B.EARN_ERR_INVALID_ARG
    assert dec(m, layer=0) == B.EARN_ERR_INVALID_ARG                                 # a full layer needs the prompt K/V
    assert dec(m, q=0) == B.EARN_ERR_INVALID_ARG
    assert dec(m, q=0x1008) == B.EARN_ERR_INVALID_ARG
    assert dec(m, cache=B.make_cache(0x1000, 0x1000, None, 1, 4, 0x1000, 0x1000, None, 1, 4, None)) == B.EARN_ERR_INVALID_ARG
    assert dec(m, cache=B.make_cache(0x1000, 0x1000, None, 2, 4, 0x1000, 0x1000, None, 0, 4, None)) == B.EARN_ERR_INVALID_ARG
    assert dec(m, batch=FakeBatch([], 0, 0, max_seqlen=0)) == B.EARN_OK               # empty batch: nothing to do
    assert lib.earn_launch_count() == n0


def test_host_validation_beam_topk(lib):
    def call(batch=2, beams=4, n_live=4, vocab=100, lp=0x1000, scores=0x2000, new=0x3000, ws=0x4000, ws_bytes=1 << 20):
        return lib.earn_beam_topk(batch, beams, n_live, vocab, lp, scores, 0x5000, 0x6000, new, ws, ws_bytes, None)

    n0 = lib.earn_launch_count()
    assert call(beams=0) == B.EARN_ERR_INVALID_ARG
    assert call(beams=33) == B.EARN_ERR_INVALID_ARG
    assert call(n_live=0) == B.EARN_ERR_INVALID_ARG
    assert call(n_live=5) == B.EARN_ERR_INVALID_ARG
    assert call(beams=4, n_live=1, vocab=3) == B.EARN_ERR_INVALID_ARG      # three continuations cannot fill four beams
    assert call(lp=0) == B.EARN_ERR_INVALID_ARG
    assert call(lp=0x1002) == B.EARN_ERR_INVALID_ARG                        # fp32 pointers are 4-byte aligned
    assert call(new=0x2000) == B.EARN_ERR_INVALID_ARG                       # the new scores would overwrite the old in place
    assert call(ws=0) == B.EARN_ERR_WORKSPACE
    assert call(beams=20, n_live=20, vocab=152064, ws_bytes=256) == B.EARN_ERR_WORKSPACE
    assert call(beams=32, n_live=32, vocab=1 << 26) == B.EARN_ERR_UNSUPPORTED   # flat candidate indices are 32-bit
    assert call(batch=0) == B.EARN_OK
    assert lib.earn_launch_count() == n0
    # one chunk needs no partial lists; 20 beams x 152064 tokens = 372 chunks of 8192 candidates, 20 (score, index) pairs each
    assert lib.earn_beam_topk_workspace_bytes(48, 20, 100) == 256
    assert lib.earn_beam_topk_workspace_bytes(48, 20, 152064) >= 48 * 372 * 20 * 8


def test_host_validation_register_qkv(lib):
    m = B.make_model(4, 2, 8, 2, 128, "bf16")
    b = FakeBatch([40, 50], 10, 10)
    cache = B.make_cache(0x1000, 0x1000, None, 2, 4, 0x1000, 0x1000, None, 1, 4, None)

    def proj(d_model=512, max_pos=64, eps=1e-6, cos=0x1000):
        return B.EarnProj(d_model, max_pos, eps, 0, cos, 0x1000)

    def call(layer=2, p=None, model=m, x=0x1000, ws=0x1000, scratch=0x1000):
        p = p or proj()
        return lib.earn_register_qkv(C.byref(model), C.byref(b.c), layer, C.byref(p), x, 0x1000, 0x1000, scratch,
                                     C.byref(cache), 0x1000, ws, 1 << 20, None)

    assert call(layer=1) == B.EARN_ERR_INVALID_ARG                       # a full layer has no register projection
    assert call(p=proj(d_model=520)) == B.EARN_ERR_INVALID_ARG           # not a multiple of 64
    assert call(p=proj(max_pos=49)) == B.EARN_ERR_INVALID_ARG            # a 50-token prompt needs 50 table rows
    assert call(p=proj(eps=-1.0)) == B.EARN_ERR_INVALID_ARG
    assert call(p=proj(cos=None)) == B.EARN_ERR_INVALID_ARG
    assert call(x=0x1008) == B.EARN_ERR_INVALID_ARG                      # 16-byte alignment
    assert call(scratch=None) == B.EARN_ERR_INVALID_ARG
    assert call(ws=0) == B.EARN_ERR_WORKSPACE
    assert call(model=B.make_model(4, 2, 8, 2, 128, "f32")) == B.EARN_ERR_UNSUPPORTED
    assert call(model=B.make_model(4, 2, 8, 2, 64, "bf16")) == B.EARN_ERR_UNSUPPORTED


def test_workspace_size_covers_the_decode_partials(lib):
    m = B.make_model(32, 8, 32, 8, 128, "bf16")
    b = FakeBatch([4096] * 8, 16, 16)
    need = lib.earn_workspace_bytes(C.byref(m), C.byref(b.c), 1)
    # 64 (sequence, kv head) units must be split several ways to fill 148 SMs: the partials
    # ([B, Hkv, splits, 16 rows, D + 1] fp32) dominate the workspace
    assert 64 * 4 * 16 * 129 * 4 < need < 64 * 64 * 16 * 129 * 4
    assert lib.earn_workspace_bytes(C.byref(m), C.byref(b.c), 0) == 256   # bad beam width -> only the status word
