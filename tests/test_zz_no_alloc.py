"""The allocation-free windowed attention entry point against the workspace-based one.

Some users of this library cannot allocate device memory for a workspace: they run inside a runtime
that owns the allocator, or under a memory budget fixed at start-up. wmtp_draft_attn_windowed_noalloc
serves them from a fixed scratch array inside the library; it must give the same result as
wmtp_draft_attn_windowed, call after call, although the array is shared and keeps old contents.
Collected last on purpose (file name), so a stop-at-first-failure run has finished every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2607_21535_b200 as wm
import wmtp_inputs as wi

from harness import DeviceWorkload

pytestmark = pytest.mark.gpu


def _cfg(**kw):
    base = dict(name="noalloc", batch=2, S0=0, S0_range=(300, 3000), Hq=16, Hkv=2, D=256, W=512, n_sink=4, gamma=2,
                seed=2024)
    base.update(kw)
    return wi.DraftConfig(**base)


@pytest.mark.parametrize("D", [256, 128])
def test_noalloc_matches_workspace_entry_point_twice_in_a_row(D):
    wm.wmtp_set_max_ctas(0)
    cfg = _cfg(D=D)
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    wm.wmtp_ring_init_from_kv(dw.ring, dw.kv)
    shape = (cfg.batch, cfg.Hq, cfg.D)
    for i in range(cfg.gamma):                                   # two calls in a row, ring advanced in between
        wm.wmtp_ring_append(dw.ring, dw.k_new[i], dw.v_new[i])
        ref = torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        ref_lse = torch.full(shape[:2], float("nan"), device="cuda")
        got = torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        got_lse = torch.full(shape[:2], float("nan"), device="cuda")
        wm.wmtp_draft_attn_windowed(dw.q[i], dw.ring, ref, dw.ws, lse=ref_lse)
        wm.wmtp_draft_attn_windowed_noalloc(dw.q[i], dw.ring, got, lse=got_lse)
        torch.cuda.synchronize()
        assert torch.isfinite(got.float()).all()
        d = (got.float() - ref.float()).abs()
        assert d.max().item() <= 2e-2 and d.mean().item() <= 2e-3          # the tolerance of the parity tests
        assert (got_lse - ref_lse).abs().max().item() <= 1e-3
        # same kernels on the same bits: equal up to the order in which split-KV partials are summed
        assert d.max().item() <= 4e-3


def test_noalloc_rejects_shapes_beyond_its_scratch():
    ring = wm.Ring(17, 2, 128, 4, 64)                            # 34 (sequence, KV head) pairs > 32
    q = torch.zeros((17, 16, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(q)
    with pytest.raises(wm.WmtpError) as ei:
        wm.wmtp_draft_attn_windowed_noalloc(q, ring, out)
    assert ei.value.status == 3 and "workspace" in str(ei.value)
    with pytest.raises(wm.WmtpError) as ei:
        wm.wmtp_draft_attn_windowed_noalloc(q[:1], wm.Ring(1, 2, 128, 4, 64), None)
    assert ei.value.status == 1
