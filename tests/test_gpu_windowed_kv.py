"""Windowed draft attention read straight from the KV store (the paper's reduced-block-table mechanism, Section 4;
Appendix A pseudocode) against the oracle's list-based sink + window store, on the same seeded bits."""
import numpy as np
import pytest
import torch

import paper_2607_21535_b200 as wm
import wmtp_inputs as wi
from oracle import reference as R

from harness import DeviceWorkload, bits, compare, oracle_for

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _defaults():
    wm.wmtp_set_max_ctas(0)
    wm.wmtp_set_work_stealing(True)
    yield
    wm.wmtp_set_max_ctas(0)


def _cfg(**kw):
    base = dict(name="wkv", batch=1, S0=300, Hq=16, Hkv=2, D=128, W=64, n_sink=4, gamma=3, seed=555)
    base.update(kw)
    return wi.DraftConfig(**base)


def _run(cfg, max_ctas=0, seqs=None):
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    wm.wmtp_set_max_ctas(max_ctas)
    out = torch.full_like(dw.q, float("nan"))
    lse = torch.full(dw.q.shape[:-1], float("nan"), dtype=torch.float32, device="cuda")
    wm.wmtp_draft_loop_windowed_kv(dw.kv, cfg.n_sink, cfg.W, dw.q, dw.k_new, dw.v_new, out, dw.ws, lse=lse)
    wm.wmtp_device_status(dw.ws)
    assert (dw.lens.cpu().numpy() == wl.seq_lens + cfg.gamma).all()
    for b in (range(cfg.batch) if seqs is None else seqs):
        orc = oracle_for(wl, b, with_ring=False)
        for i in range(cfg.gamma):
            r = orc.step(wl.q[i, b], wl.k_new[i, b], wl.v_new[i, b], full=False)
            compare(out[i, b], lse[i, b], *r["win"], what=f"{cfg.name} ctas={max_ctas} seq={b} step={i}")
    return dw, wl


@pytest.mark.parametrize("paged", [False, True])
@pytest.mark.parametrize("D", [128, 256])
@pytest.mark.parametrize("S0", [0, 1, 3, 4, 60, 62, 63, 64, 65, 66, 67, 68, 130, 200, 1000])
def test_window_view_all_boundaries(paged, D, S0):
    # n_sink + W = 68; the three appends walk S across sink-only, page-boundary, exactly-full and sliding states
    _run(_cfg(S0=S0, D=D, paged=paged, seed=700 + S0))


@pytest.mark.parametrize("n_sink,W", [(0, 1), (0, 64), (1, 1), (70, 100), (64, 64), (4, 129), (130, 7)])
@pytest.mark.parametrize("S0", [5, 150, 777])
def test_window_view_sink_and_window_sizes(n_sink, W, S0):
    _run(_cfg(S0=S0, n_sink=n_sink, W=W, paged=True, seed=S0 + n_sink))
    _run(_cfg(S0=S0, n_sink=n_sink, W=W, D=256, seed=S0 + W), max_ctas=3)


def test_window_view_appends_land_in_the_store_bit_exact():
    cfg = _cfg(S0=500, paged=True, gamma=4, batch=3, S0_range=(100, 900), seed=12)
    dw, wl = _run(cfg)
    Kd = bits(dw.K)
    for b in range(cfg.batch):
        for i in range(cfg.gamma):
            p = int(wl.seq_lens[b]) + i
            page = wl.page_table[b, p // 64]
            assert (Kd[page, :, p % 64] == wl.k_new[i, b]).all()


def test_window_view_equals_ring_path():
    cfg = _cfg(S0=20000, D=256, W=2048, gamma=2, seed=3)
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    dw.run_loops(full=False)                               # ring path
    dw2 = DeviceWorkload(wl)
    out = torch.empty_like(dw2.q)
    lse = torch.empty(dw2.q.shape[:-1], dtype=torch.float32, device="cuda")
    wm.wmtp_draft_loop_windowed_kv(dw2.kv, cfg.n_sink, cfg.W, dw2.q, dw2.k_new, dw2.v_new, out, dw2.ws, lse=lse)
    wm.wmtp_device_status(dw2.ws)
    assert (out.float() - dw.out_w.float()).abs().max().item() <= 4e-3
    assert (lse - dw.lse_w).abs().max().item() <= 1e-4


def test_window_view_batched_paged_ragged():
    cfg = wi.scaled(wi.CONFIGS[3], batch=6, S0_range=(2048, 65536), gamma=3, name="wkv_batched")
    _run(cfg)


def test_window_view_million_token_context():
    _run(wi.scaled(wi.CONFIGS[2], gamma=2, name="wkv_million"))


def test_window_view_rejects_bad_window():
    cfg = _cfg(S0=10)
    dw = DeviceWorkload(wi.make_workload(cfg))
    out = torch.empty_like(dw.q[0])
    with pytest.raises(wm.WmtpError) as ei:
        wm.wmtp_draft_attn_windowed_kv(dw.q[0], dw.kv, 4, 0, out, dw.ws)
    assert ei.value.status == 1


@pytest.mark.parametrize("kv_dtype,D", [("fp8", 128), ("fp8", 256), ("bf16", 128)])
@pytest.mark.parametrize("paged", [False, True])
def test_window_view_long_enough_for_the_streaming_form(kv_dtype, D, paged):
    """A window of 40000 tokens is served by the cooperative (streaming) form: with an fp8 head_dim-128 store its tiles
    travel in pairs, and with three sink tiles (n_sink = 130) one pair holds the last sink tile and the first window
    tile -- rows from two places of the store, each with its own row bounds."""
    cfg = _cfg(S0=90001, n_sink=130, W=40000, D=D, Hq=8, Hkv=1, gamma=2, paged=paged, seed=611, kv_dtype=kv_dtype)
    _run(cfg)
    _run(cfg, max_ctas=5)


# ------------------------------------------------------------------------------------------ the reduced block table itself
@pytest.mark.parametrize("n_sink,W", [(4, 64), (0, 100), (64, 252), (70, 130), (4, 2048)])
def test_reduced_block_table_bit_exact(n_sink, W):
    cfg = wi.DraftConfig("rbt", 9, 0, 16, 2, 128, W, n_sink, 1, seed=1000 + W, S0_range=(n_sink + W + 2, 9000), paged=True)
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    lens = wl.seq_lens.copy()
    # shorter than generated (the pages exist): empty, sink only, partly filled window, exactly full, first slide
    lens[0], lens[1], lens[2], lens[3], lens[4] = 0, max(n_sink - 1, 1), n_sink + W // 2, n_sink + W, n_sink + W + 1
    dw.lens.copy_(torch.from_numpy(lens))
    width = wm.wmtp_reduced_block_table_width(n_sink, W, 64)
    assert width == (n_sink + 63) // 64 + (W + 63) // 64 + 1
    table = torch.full((cfg.batch, width + 2), -7, dtype=torch.int32, device="cuda")
    meta = torch.full((cfg.batch, 5), -7, dtype=torch.int32, device="cuda")
    wm.wmtp_reduced_block_table(dw.kv, n_sink, W, table, meta, dw.ws)
    wm.wmtp_device_status(dw.ws)
    tb, mt = table.cpu().numpy(), meta.cpu().numpy()
    for b in range(cfg.batch):
        S = int(lens[b])
        pages, m = R.reduced_block_table(S, n_sink, W, wl.page_table[b], 64)
        assert mt[b].tolist() == m, (b, S)
        assert tb[b, :len(pages)].tolist() == pages and (tb[b, len(pages):] == -1).all()


def test_reduced_block_table_needs_a_wide_enough_table_and_a_paged_store():
    cfg = wi.DraftConfig("rbt2", 2, 500, 16, 2, 128, 256, 4, 1, seed=7, paged=True)
    dw = DeviceWorkload(wi.make_workload(cfg))
    meta = torch.zeros((2, 5), dtype=torch.int32, device="cuda")
    with pytest.raises(wm.WmtpError) as ei:
        wm.wmtp_reduced_block_table(dw.kv, 4, 256, torch.zeros((2, 5), dtype=torch.int32, device="cuda"), meta)
    assert ei.value.status == 3
    dc = DeviceWorkload(wi.make_workload(wi.scaled(cfg, paged=False)))
    with pytest.raises(wm.WmtpError) as ei:
        wm.wmtp_reduced_block_table(dc.kv, 4, 256, torch.zeros((2, 8), dtype=torch.int32, device="cuda"), meta)
    assert ei.value.status == 1


# ------------------------------------------------------------------------------------------ the O(S) counterpart
def test_full_token_index_bit_exact_and_flags_a_short_table():
    cfg = wi.DraftConfig("fti", 7, 0, 16, 2, 128, 64, 4, 1, seed=77, S0_range=(1, 9000), paged=True)
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    lens = wl.seq_lens.copy()
    lens[0], lens[1], lens[2] = 0, 1, 64
    dw.lens.copy_(torch.from_numpy(lens))
    stride = int(lens.max()) + 37
    index = dw.guard((cfg.batch, stride), torch.int32, "cuda", "the token index").fill_(-7)
    wm.wmtp_full_token_index(dw.kv, index, dw.ws)
    wm.wmtp_device_status(dw.ws)
    dw.guard.check("token index")
    got = index.cpu().numpy()
    for b in range(cfg.batch):
        assert got[b].tolist() == R.full_token_index(int(lens[b]), wl.page_table[b], 64, stride), b
    # a table shorter than the longest sequence: its entries are still right, the overflow is flagged
    short = torch.full((cfg.batch, 100), -7, dtype=torch.int32, device="cuda")
    wm.wmtp_full_token_index(dw.kv, short, dw.ws)
    with pytest.raises(wm.WmtpError) as ei:
        wm.wmtp_device_status(dw.ws)
    assert ei.value.status == 7
    sh = short.cpu().numpy()
    for b in range(cfg.batch):
        assert sh[b].tolist() == R.full_token_index(int(lens[b]), wl.page_table[b], 64, 100)
    dc = DeviceWorkload(wi.make_workload(wi.scaled(cfg, paged=False, S0=300, S0_range=None)))
    with pytest.raises(wm.WmtpError) as ei:
        wm.wmtp_full_token_index(dc.kv, short)
    assert ei.value.status == 1
