"""The C-ABI library loads without a GPU, exports every symbol the header declares, and rejects
bad arguments on the host before anything is launched."""
import ctypes
import os
import re

import pytest

import paper_2607_21535_b200 as wm
from paper_2607_21535_b200 import binding, build as wbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    wbuild.build()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "wmtp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(wmtp_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    names = _declared_symbols()
    assert len(names) >= 18
    L = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(L, n), f"{n} declared in wmtp.h but not exported"
        assert n in binding._SIGNATURES, f"{n} has no ctypes signature"
        assert hasattr(wm, n), f"{n} has no Python binding of the same name"
    assert sorted(binding._SIGNATURES) == names


def test_sizes():
    kb, pb = wm.wmtp_ring_bytes(1, 2, 256, 4, 4096)
    assert kb == 2 * 4100 * 256 * 2 and pb == 4100 * 4
    assert wm.wmtp_ring_bytes(0, 2, 256, 4, 4096) == (0, 0)
    ws = wm.wmtp_workspace_bytes(1, 16, 2, 256)
    assert ws % 256 == 0 and ws > 148 * 8 * 257 * 4
    assert wm.wmtp_workspace_bytes(1, 15, 2, 256) == 0
    assert wm.wmtp_stage_bytes(7, 1, 16, 2, 256) >= 7 * (2 * 16 * 256 * 2 + 2 * 2 * 256 * 2)
    assert wm.wmtp_status_string(0) == "ok" and "bounds" in wm.wmtp_status_string(7)


def test_ring_snapshot_size_and_arguments_rejected_on_host():
    L = wm.lib()
    good = _ring_desc()
    # K and V rows (2 KV heads x 12 slots x 128 x 2 bytes), slot_pos (12 x 4), len (8): each part on a 256-byte boundary
    assert L.wmtp_ring_state_bytes(ctypes.byref(good)) == 2 * 6144 + 256 + 256
    f8 = _ring_desc(kv_dtype=1, k_scale=4096, v_scale=4096)
    assert L.wmtp_ring_state_bytes(ctypes.byref(f8)) == 2 * 3072 + 256 + 256
    assert L.wmtp_ring_state_bytes(ctypes.byref(_ring_desc(W=0))) == 0
    need = L.wmtp_ring_state_bytes(ctypes.byref(good))
    for fn in (L.wmtp_ring_export, L.wmtp_ring_import):
        assert fn(ctypes.byref(good), None, need, None) == 1                       # no blob
        assert fn(ctypes.byref(good), 4104, need, None) == 1                       # misaligned blob
        assert fn(ctypes.byref(good), 4096, need - 1, None) == 3                   # blob too small
        assert "takes" in wm.wmtp_last_error()
        assert fn(ctypes.byref(_ring_desc(cap=4)), 4096, need, None) == 1          # bad descriptor


def _ring_desc(**kw):
    d = dict(k=4096, v=8192, slot_pos=4096, len=4096, batch=1, Hkv=2, D=128, n_sink=4, W=8, cap=8)
    d.update(kw)
    return binding.wmtp_ring(**d)


def _kv_desc(**kw):
    d = dict(k=4096, v=8192, page_table=None, len=4096, S_cap=100, batch=1, Hkv=2, D=128, page_size=0, max_pages=0,
             num_pages=0)
    d.update(kw)
    return binding.wmtp_kv(**d)


@pytest.mark.parametrize("kw,status", [
    (dict(k=None), 1), (dict(k=4100), 1), (dict(W=0), 1), (dict(cap=4), 1), (dict(n_sink=-1), 1),
    (dict(D=64), 2), (dict(batch=0), 1), (dict(batch=5000), 2), (dict(len=None), 1),
])
def test_ring_descriptor_rejected_on_host(kw, status):
    L = wm.lib()
    r = _ring_desc(**kw)
    assert L.wmtp_ring_reset(ctypes.byref(r), None) == status
    assert L.wmtp_ring_append(ctypes.byref(r), 4096, 4096, None) == status
    assert wm.wmtp_last_error() != ""


@pytest.mark.parametrize("kw,status", [
    (dict(v=None), 1), (dict(S_cap=0), 1), (dict(D=96), 2),
    (dict(page_table=4096, page_size=16, max_pages=4, num_pages=8), 2),
    (dict(page_table=4096, page_size=64, max_pages=1, num_pages=8, S_cap=100), 3),
    (dict(page_table=4098, page_size=64, max_pages=4, num_pages=8), 1),
])
def test_kv_descriptor_rejected_on_host(kw, status):
    L = wm.lib()
    kv = _kv_desc(**kw)
    assert L.wmtp_kv_append(ctypes.byref(kv), 4096, 4096, None, None) == status
    assert L.wmtp_draft_attn_full(4096, 16, ctypes.byref(kv), 0.0, 4096, None, 4096, 1 << 30, None) == status


def test_attention_arguments_rejected_on_host():
    L = wm.lib()
    r, kv = _ring_desc(), _kv_desc()
    big = 1 << 30
    assert L.wmtp_draft_attn_windowed(None, 16, ctypes.byref(r), 0.0, 4096, None, 4096, big, None) == 1
    assert L.wmtp_draft_attn_windowed(4096, 15, ctypes.byref(r), 0.0, 4096, None, 4096, big, None) == 1
    assert L.wmtp_draft_attn_windowed(4096, 32, ctypes.byref(r), 0.0, 4096, None, 4096, big, None) == 2   # group of 16
    assert L.wmtp_draft_attn_windowed(4096, 16, ctypes.byref(r), 0.0, 4096, None, None, big, None) == 4
    assert L.wmtp_draft_attn_windowed(4096, 16, ctypes.byref(r), 0.0, 4096, None, 4096 + 64, big, None) == 4
    assert L.wmtp_draft_attn_windowed(4096, 16, ctypes.byref(r), 0.0, 4096, None, 4096, 1000, None) == 4
    assert L.wmtp_draft_attn_full(4096, 16, ctypes.byref(kv), 0.0, None, None, 4096, big, None) == 1
    assert L.wmtp_draft_loop_full(ctypes.byref(kv), 0, 4096, 16, 4096, 4096, 0.0, 4096, None, 4096, big, None) == 1
    assert L.wmtp_draft_loop_windowed(ctypes.byref(r), 3, 4096, 16, None, 4096, 0.0, 4096, None, 4096, big, None) == 1
    assert L.wmtp_workspace_init(None, 4096, None) == 4
    assert L.wmtp_ring_init_from_kv(ctypes.byref(r), ctypes.byref(_kv_desc(Hkv=4)), None) == 1
    with pytest.raises(wm.WmtpError):
        binding._check(1)


def test_extend_and_rollback_arguments_rejected_on_host():
    L = wm.lib()
    r, kv = _ring_desc(cap=12), _kv_desc()
    big = 1 << 30
    rb, kb = ctypes.byref(r), ctypes.byref(kv)
    assert L.wmtp_draft_extend_windowed(4096, 0, 16, rb, 0.0, 4096, None, 4096, big, None) == 1       # q_len < 1
    assert L.wmtp_draft_extend_windowed(4096, 65, 16, rb, 0.0, 4096, None, 4096, big, None) == 1      # q_len > 64
    assert L.wmtp_draft_extend_windowed(4096, 6, 16, rb, 0.0, 4096, None, 4096, big, None) == 3       # cap 12 < W + 5
    assert L.wmtp_draft_extend_windowed(None, 5, 16, rb, 0.0, 4096, None, 4096, big, None) == 1
    assert L.wmtp_draft_extend_windowed(4096, 5, 16, rb, 0.0, 4096, None, 4096, 1000, None) == 4      # workspace too small
    assert L.wmtp_draft_extend_full(4096, 0, 16, kb, 0.0, 4096, None, 4096, big, None) == 1
    assert L.wmtp_draft_extend_full(4096, 4, 16, ctypes.byref(_kv_desc(batch=512)), 0.0, 4096, None, 4096, big, None) == 2
    assert L.wmtp_draft_extend_full(4096, 4, 16, kb, 0.0, None, None, 4096, big, None) == 1
    assert L.wmtp_ring_append_many(rb, 0, 4096, 4096, None) == 1
    assert L.wmtp_ring_append_many(rb, 3, None, 4096, None) == 1
    assert L.wmtp_kv_append_many(kb, 0, 4096, 4096, None, None) == 1
    assert L.wmtp_kv_append_many(kb, 2, 4096, None, None, None) == 1
    assert L.wmtp_ring_rewind(rb, None, None, None) == 1
    assert L.wmtp_ring_rewind(ctypes.byref(_ring_desc(W=0)), 4096, None, None) == 1


def test_kv_dtype_rejected_on_host():
    L = wm.lib()
    assert wm.wmtp_kv_elem_bytes(0) == 2 and wm.wmtp_kv_elem_bytes(1) == 1 and wm.wmtp_kv_elem_bytes(5) == 0
    # an fp8 store without scales, or with misaligned ones
    assert L.wmtp_ring_reset(ctypes.byref(_ring_desc(kv_dtype=1)), None) == 1
    assert L.wmtp_ring_reset(ctypes.byref(_ring_desc(kv_dtype=1, k_scale=4096, v_scale=4098)), None) == 1
    assert L.wmtp_kv_append(ctypes.byref(_kv_desc(kv_dtype=1, k_scale=4096)), 4096, 4096, None, None) == 1
    # an unknown entry type
    assert L.wmtp_ring_reset(ctypes.byref(_ring_desc(kv_dtype=2, k_scale=4096, v_scale=4096)), None) == 2
    assert L.wmtp_draft_attn_full(4096, 16, ctypes.byref(_kv_desc(kv_dtype=9)), 0.0, 4096, None, 4096, 1 << 30, None) == 2
    # rows are copied as stored: ring and KV store must agree
    r8 = _ring_desc(kv_dtype=1, k_scale=4096, v_scale=4096)
    assert L.wmtp_ring_init_from_kv(ctypes.byref(r8), ctypes.byref(_kv_desc()), None) == 1


def test_reduced_block_table_arguments_rejected_on_host():
    L = wm.lib()
    paged = _kv_desc(page_table=4096, page_size=64, max_pages=4, num_pages=8, S_cap=256)
    assert wm.wmtp_reduced_block_table_width(4, 64, 64) == 3 and wm.wmtp_reduced_block_table_width(64, 4032, 64) == 65
    assert wm.wmtp_reduced_block_table_width(-1, 64, 64) == 0
    assert L.wmtp_reduced_block_table(ctypes.byref(paged), 4, 64, 4096, 2, 4096, None, None) == 3      # needs 3 entries
    assert L.wmtp_reduced_block_table(ctypes.byref(paged), 4, 0, 4096, 8, 4096, None, None) == 1
    assert L.wmtp_reduced_block_table(ctypes.byref(paged), 4, 64, None, 8, 4096, None, None) == 1
    assert L.wmtp_reduced_block_table(ctypes.byref(_kv_desc()), 4, 64, 4096, 8, 4096, None, None) == 1  # contiguous store
