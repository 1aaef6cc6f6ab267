"""Seeded random shapes through the whole path (fused draft loops, windowed and full-context, every store type and
layout, CTA caps, stealing on and off) against the oracle: a sweep over the corners the targeted tests do not name."""
import numpy as np
import pytest
import torch

import paper_2607_21535_b200 as wm
import wmtp_inputs as wi

from harness import DeviceWorkload, check_ring_against_sim, compare, oracle_for

pytestmark = pytest.mark.gpu


def _random_cfg(rs, idx):
    D = int(rs.choice([128, 256]))
    Hkv = int(rs.choice([1, 2, 4]))
    G = int(rs.choice([1, 2, 4, 7, 8]))
    batch = int(rs.choice([1, 1, 2, 3, 5, 9]))
    hi = int(rs.choice([300, 3000, 20000, 60000]))
    n_sink = int(rs.choice([0, 1, 4, 64, 70]))
    W = int(rs.choice([1, 17, 64, 200, 1024, 4096]))
    return wi.DraftConfig(
        name=f"rand{idx}", batch=batch, S0=0, Hq=G * Hkv, Hkv=Hkv, D=D, W=W, n_sink=n_sink, gamma=int(rs.choice([1, 2, 4])),
        seed=7000 + idx, S0_range=(1, hi), paged=bool(rs.randint(2)), cap_slack=int(rs.choice([0, 0, 3, 9])),
        kv_dtype=str(rs.choice(["bf16", "fp8"])), key_scale=(0.5, 2.0) if Hkv > 1 and rs.randint(2) else None)


@pytest.mark.parametrize("idx", range(36))
def test_random_shape(idx):
    rs = np.random.RandomState(9000 + idx)
    cfg = _random_cfg(rs, idx)
    max_ctas = int(rs.choice([0, 0, 0, 1, 3, 11, 64, 147]))
    stealing = bool(rs.randint(4))                     # mostly on
    wm.wmtp_set_max_ctas(max_ctas)
    wm.wmtp_set_work_stealing(stealing)
    try:
        wl = wi.make_workload(cfg)
        dw = DeviceWorkload(wl)
        dw.run_loops()
        # the same windowed steps read straight from a second copy of the KV store (window view), loop form
        dv = DeviceWorkload(wl)
        out_v, lse_v = torch.full_like(dv.q, float("nan")), torch.full_like(dv.lse_w, float("nan"))
        wm.wmtp_draft_loop_windowed_kv(dv.kv, cfg.n_sink, cfg.W, dv.q, dv.k_new, dv.v_new, out_v, dv.ws, lse=lse_v)
        wm.wmtp_device_status(dv.ws)
        seqs = sorted(set([0, cfg.batch - 1, int(np.argmax(wl.seq_lens)), int(np.argmin(wl.seq_lens))]))
        for b in seqs:
            orc = oracle_for(wl, b)
            for i in range(cfg.gamma):
                r = orc.step(wl.q[i, b], wl.k_new[i, b], wl.v_new[i, b])
                tag = f"{cfg} ctas={max_ctas} stealing={stealing} seq={b} step={i}"
                compare(dw.out_w[i, b], dw.lse_w[i, b], *r["win"], what=tag + " windowed")
                compare(dw.out_f[i, b], dw.lse_f[i, b], *r["full"], what=tag + " full")
                compare(out_v[i, b], lse_v[i, b], *r["win"], what=tag + " window view")
            check_ring_against_sim(dw.ring, b, orc.ring, f"{cfg} seq={b}")
            assert int(dw.lens[b]) == orc.S
    finally:
        wm.wmtp_set_max_ctas(0)
        wm.wmtp_set_work_stealing(True)
