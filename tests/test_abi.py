"""Host-side checks of the C boundary (no GPU needed): the library builds, loads and exports every symbol the
header declares, and argument validation rejects bad calls before anything is launched."""
import ctypes
import os
import re

import pytest

from paper_2609_36938_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "janus.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(janus_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    declared = _declared_symbols()
    assert len(declared) >= 10
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in janus.h but not exported"
    assert sorted(binding.EXPORTS) == declared


def test_version_and_workspace_queries(lib):
    assert lib.janus_version() >= 100
    assert lib.janus_indexer_scores_workspace_size(16, 64, 128, 4096, 0) == 0
    assert lib.janus_topk_workspace_size(16, 4096, 64) == 0
    assert lib.janus_page_demand_workspace_size(16, 64, 100) == 0
    assert lib.janus_sparse_attn_prefill_workspace_size(16, 128, 576, 512, 64) == 0


def test_invalid_arguments_are_rejected_on_the_host(lib):
    INVALID, UNSUPPORTED = 1, 2
    fake = ctypes.c_void_p(0x1000)       # aligned, never dereferenced: validation fails first
    odd = ctypes.c_void_p(0x1004)
    # indexer: bad dtype, D not a multiple of 16, NULL pointers, misaligned pointer, scores_ld too small, fp8 without scales
    args = dict(q=fake, qs=64 * 128, k=fake, ks=128, w=fake, qsc=None, qss=0, ksc=None, rb=None, cb=None, M=4, H=64, D=128, n=256,
                pos=0, causal=1, dt=0, sc=fake, ld=256)

    def idx_call(**kw):
        a = dict(args, **kw)
        return lib.janus_indexer_scores(a["q"], a["qs"], a["k"], a["ks"], a["w"], a["qsc"], a["qss"], a["ksc"], a["rb"], a["cb"], a["M"],
                                        a["H"], a["D"], a["n"], a["pos"], a["causal"], a["dt"], a["sc"], a["ld"], None, 0, None, None)

    assert idx_call(dt=7) == UNSUPPORTED
    assert idx_call(D=100) == UNSUPPORTED
    assert idx_call(q=None) == INVALID
    assert idx_call(q=odd) == INVALID
    assert idx_call(ld=100) == INVALID
    assert idx_call(ld=258) == INVALID
    assert idx_call(dt=1) == INVALID                      # fp8 needs both scale arrays
    assert idx_call(rb=fake) == INVALID                   # bias factors come in pairs
    assert idx_call(M=-1) == INVALID
    assert idx_call(M=0) == 0                             # nothing to do
    # top-k
    assert lib.janus_topk(fake, 256, 4, 256, 0, 1, 0, fake, None, None, None, 0, None, None) == INVALID      # k = 0
    assert lib.janus_topk(fake, 100, 4, 256, 0, 1, 8, fake, None, None, None, 0, None, None) == INVALID      # ld < n_keys
    assert lib.janus_topk(odd, 256, 4, 256, 0, 1, 8, fake, None, None, None, 0, None, None) == INVALID       # misaligned
    assert lib.janus_topk(fake, 256, 4, 256, 0, 1, 8, None, None, None, None, 0, None, None) == INVALID      # no output
    assert lib.janus_topk(fake, 256, 0, 256, 0, 1, 8, fake, None, None, None, 0, None, None) == 0            # M = 0
    # page demand: page_size 0, missing outputs, partial miss group
    def pd(page_size=64, bitmap=fake, miss=(None, None, None, None), n_phys=64):
        return lib.janus_page_demand(fake, 4, 8, 100, page_size, fake, 4, n_phys, None, bitmap, fake, fake, fake, fake, *miss, 64,
                                     None, 0, None, None)
    assert pd(page_size=0) == INVALID
    assert pd(bitmap=None) == INVALID
    assert pd(miss=(fake, None, None, None)) == INVALID
    assert pd(n_phys=0) == INVALID
    # attention: head counts that do not divide, unsupported dims, misaligned strides
    def at(H_q=8, n_kv=8, d_qk=128, d_v=128, tok_stride=1024, q=fake):
        return lib.janus_sparse_attn_prefill(q, 4, H_q, d_qk, fake, fake, 65536, tok_stride, 128, n_kv, d_v, fake, 16, 64, fake, 4,
                                             ctypes.c_float(1.0), fake, None, None, 0, None, None)
    assert at(H_q=6, n_kv=4) == INVALID
    assert at(d_qk=132) == UNSUPPORTED
    assert at(d_v=1024) == UNSUPPORTED
    assert at(tok_stride=1001) == INVALID
    assert at(q=None) == INVALID
    assert at(d_qk=64, d_v=128) == INVALID                # k_pool == v_pool here: an aliased value row cannot be wider than the key row


def test_binding_refuses_host_tensors_and_missing_library(monkeypatch):
    import torch

    with pytest.raises(binding.JanusError):
        binding._ptr(torch.zeros(4))
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libjanus.so")
    with pytest.raises(binding.JanusError):
        binding.load()


def test_batch_entry_and_static_entry_validation(lib):
    """Host-side rejection for the entry points added after the four basic calls (nothing is launched on these paths)."""
    INVALID, UNSUPPORTED, TOO_SMALL = 1, 2, 3
    fake = ctypes.c_void_p(0x1000)
    # decode batch: missing offsets, max_keys beyond the key array, head count the ragged tensor-core mode does not take
    sb = lambda **kw: lib.janus_indexer_scores_batch(kw.get("q", fake), fake, 128, fake, None, 0, None, None, None, kw.get("B", 4), kw.get("H", 64),
                                                      128, kw.get("off", fake), 4096, kw.get("max_keys", 1024), 0, kw.get("sc", fake), None, None)
    assert sb(off=None) == INVALID
    assert sb(max_keys=5000) == INVALID
    assert sb(sc=None) == INVALID
    assert sb(H=32) == UNSUPPORTED
    assert sb(B=0) == 0
    assert lib.janus_topk_batch(fake, fake, None, 4, 0, fake, None, None, None, None) == INVALID          # k = 0
    assert lib.janus_topk_batch(fake, None, None, 4, 8, fake, None, None, None, None) == INVALID          # no offsets
    assert lib.janus_topk_batch(fake, fake, None, 0, 8, fake, None, None, None, None) == 0                # empty batch
    pdb = lambda **kw: lib.janus_page_demand_batch(fake, 4, 8, kw.get("lim", fake), kw.get("page", 64), fake, kw.get("off", fake), 64, None,
                                                   kw.get("bitmap", fake), fake, fake, fake, fake, None, None, None, None, 64, None, None)
    assert pdb(page=0) == INVALID
    assert pdb(lim=None) == INVALID
    assert pdb(off=None) == INVALID
    assert pdb(bitmap=None) == INVALID
    assert lib.janus_sparse_attn_decode(fake, 4, 128, 576, fake, fake, 64 * 576, 576, 576, 1, 512, fake, 64, 64, fake, None, 0.04, fake, None,
                                        None, None) == INVALID                                              # no table offsets
    # entry granularity
    assert lib.janus_topk_entries(fake, 64, 4, 64, 0, 0, 8, fake, None, None, None, None) == INVALID       # entry_size = 0
    assert lib.janus_topk_entries(fake, 32, 4, 64, 0, 16, 8, fake, None, None, None, None) == INVALID      # ld < n_entries
    assert lib.janus_entry_expand(None, 4, 8, 16, 0, fake, None) == INVALID
    assert lib.janus_entry_pool_scores(fake, 256, 4, 256, 0, 1, 0, fake, 16, None) == INVALID               # entry_size = 0
    assert lib.janus_entry_pool_scores(fake, 256, 4, 256, 0, 1, 64, fake, 3, None) == INVALID               # entry_ld < n_entries
    assert lib.janus_entry_pool_scores(fake, 256, 4, 256, 0, 1, 64, None, 4, None) == INVALID               # no output
    assert lib.janus_entry_pool_scores(fake, 256, 0, 256, 0, 1, 64, fake, 4, None) == 0                     # M = 0
    assert lib.janus_entry_expand(fake, 0, 8, 16, 0, fake, None) == 0
    # built-in scratch: the size check comes before the device is touched
    assert lib.janus_indexer_topk_static(fake, 64 * 128, fake, 128, fake, fake, 0, fake, None, None, 4096, 64, 128, 135168, 131072, 1, 1, 2048,
                                         fake, None, None, None, None) == TOO_SMALL
    assert lib.janus_indexer_topk_static(fake, 64 * 128, fake, 128, fake, None, 0, None, None, None, 8, 64, 128, 4096, 0, 1, 0, 0,
                                         fake, None, None, None, None) == INVALID                           # k = 0
