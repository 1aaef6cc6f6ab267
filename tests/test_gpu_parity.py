"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded bits.

Ring contents, slot indices and lengths are compared bit for bit; attention outputs within
max-abs 2e-2 / mean-abs 2e-3 on the bf16 result plus a per-head relative-L2 bound of 1e-2 and an
lse bound of 1e-3 (the absolute bounds alone are nearly vacuous at large S, where outputs shrink
like 1/sqrt(S)).
"""
import math

import numpy as np
import pytest
import torch

import paper_2607_21535_b200 as wm
import wmtp_inputs as wi
from oracle import reference as R

from harness import DeviceWorkload, bits, check_ring_against_sim, compare, oracle_for, to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _default_ctas():
    wm.wmtp_set_max_ctas(0)
    wm.wmtp_set_work_stealing(True)
    yield
    wm.wmtp_set_max_ctas(0)
    wm.wmtp_set_work_stealing(True)


def _cfg(**kw):
    base = dict(name="t", batch=1, S0=300, Hq=16, Hkv=2, D=128, W=64, n_sink=4, gamma=3, seed=4321)
    base.update(kw)
    return wi.DraftConfig(**base)


# ------------------------------------------------------------------------------------------ ring store
@pytest.mark.parametrize("D", [128, 256])
@pytest.mark.parametrize("n_sink,W,cap", [(4, 8, 8), (0, 1, 1), (1, 1, 1), (2, 3, 3), (4, 8, 11), (3, 70, 70), (0, 5, 9)])
def test_ring_append_bit_exact_over_several_wraps(D, n_sink, W, cap):
    B, Hkv = 3, 2
    n = 3 * (n_sink + cap) + 5
    k = wi.normal_bf16(11, (1, D, n_sink, cap), (n, B, Hkv, D))
    v = wi.normal_bf16(11, (2, D, n_sink, cap), (n, B, Hkv, D))
    kd, vd = to_dev_bf16(k), to_dev_bf16(v)
    ring = wm.Ring(B, Hkv, D, n_sink, W, cap=cap)
    ring.k.fill_(float("nan")); ring.v.fill_(float("nan"))
    wm.wmtp_ring_reset(ring)
    sims = [R.RingSim(n_sink, cap, Hkv, D) for _ in range(B)]
    for i in range(n):
        wm.wmtp_ring_append(ring, kd[i], vd[i])
        for b in range(B):
            sims[b].append(k[i, b], v[i, b])
        if i % 7 == 0 or i == n - 1:
            for b in range(B):
                check_ring_against_sim(ring, b, sims[b], f"append {i} seq {b}")
    # never-written slots keep the reset sentinel and their bytes untouched (NaN fill)
    ring2 = wm.Ring(1, Hkv, D, n_sink, W, cap=cap)
    wm.wmtp_ring_reset(ring2)
    assert (ring2.slot_pos.cpu().numpy() == -1).all() and int(ring2.len[0]) == 0


@pytest.mark.parametrize("paged", [False, True])
@pytest.mark.parametrize("S0s", [[0, 1, 3], [4, 5, 11], [12, 13, 40], [200, 64, 129]])
@pytest.mark.parametrize("cap_slack", [0, 5])
def test_ring_bulk_init_equals_sequential_appends(paged, S0s, cap_slack):
    n_sink, W = 4, 8
    for S0 in S0s:
        cfg = _cfg(S0=S0, W=W, n_sink=n_sink, paged=paged, cap_slack=cap_slack, seed=50 + S0)
        wl = wi.make_workload(cfg)
        dw = DeviceWorkload(wl)
        wm.wmtp_ring_init_from_kv(dw.ring, dw.kv)
        sim = R.RingSim(n_sink, W + cap_slack, cfg.Hkv, cfg.D)
        for p in range(S0):
            sim.append(wl.K[0][:, p], wl.V[0][:, p])
        check_ring_against_sim(dw.ring, 0, sim, f"bulk init S0={S0}")


@pytest.mark.parametrize("paged", [False, True])
def test_kv_append_bit_exact(paged):
    cfg = _cfg(batch=3, S0=0, S0_range=(60, 200), paged=paged, gamma=5, seed=9)
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    for i in range(cfg.gamma):
        wm.wmtp_kv_append(dw.kv, dw.k_new[i], dw.v_new[i], dw.ws)
    wm.wmtp_device_status(dw.ws)
    lens = dw.lens.cpu().numpy()
    assert (lens == wl.seq_lens + cfg.gamma).all()
    Kd, Vd = bits(dw.K), bits(dw.V)
    expK, expV = wl.K_dev.copy(), wl.V_dev.copy()
    for b in range(cfg.batch):
        for i in range(cfg.gamma):
            p = int(wl.seq_lens[b]) + i
            if paged:
                page = wl.page_table[b, p // 64]
                expK[page, :, p % 64] = wl.k_new[i, b]; expV[page, :, p % 64] = wl.v_new[i, b]
            else:
                expK[b, :, p] = wl.k_new[i, b]; expV[b, :, p] = wl.v_new[i, b]
    assert (Kd == expK).all() and (Vd == expV).all()      # every other byte (NaN poison included) untouched


def test_kv_append_past_capacity_is_flagged_not_written():
    cfg = _cfg(S0=10, gamma=2)
    wl = wi.make_workload(cfg)                 # S_cap = 12
    dw = DeviceWorkload(wl)
    for i in range(2):
        wm.wmtp_kv_append(dw.kv, dw.k_new[i], dw.v_new[i], dw.ws)
    wm.wmtp_device_status(dw.ws)
    before = bits(dw.K).copy()
    wm.wmtp_kv_append(dw.kv, dw.k_new[0], dw.v_new[0], dw.ws)
    with pytest.raises(wm.WmtpError) as ei:
        wm.wmtp_device_status(dw.ws)
    assert ei.value.status == 7
    assert int(dw.lens[0]) == 12 and (bits(dw.K) == before).all()
    wm.wmtp_device_status(dw.ws)               # sticky word was cleared by the read


# ------------------------------------------------------------------------------------------ attention parity
def _run_and_check(cfg, max_ctas=0, cap=None, check_ring=True, seqs=None, steps=None):
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl, cap=cap)
    wm.wmtp_set_max_ctas(max_ctas)
    dw.run_loops()
    worst = 0.0
    for b in (range(cfg.batch) if seqs is None else seqs):
        orc = oracle_for(wl, b, cap=cap, with_ring=check_ring)
        for i in range(cfg.gamma):
            do = steps is None or i in steps
            r = orc.step(wl.q[i, b], wl.k_new[i, b], wl.v_new[i, b], full=do, windowed=do)
            if not do:
                continue
            tag = f"{cfg.name} ctas={max_ctas} seq={b} step={i}"
            e1, _ = compare(dw.out_w[i, b], dw.lse_w[i, b], *r["win"], what=tag + " windowed")
            e2, _ = compare(dw.out_f[i, b], dw.lse_f[i, b], *r["full"], what=tag + " full")
            worst = max(worst, e1, e2)
        if check_ring:
            check_ring_against_sim(dw.ring, b, orc.ring, f"{cfg.name} seq={b}")
        assert int(dw.lens[b]) == orc.S
    return worst


@pytest.mark.parametrize("D", [128, 256])
@pytest.mark.parametrize("max_ctas", [1, 2, 7, 0])
@pytest.mark.parametrize("S0", [0, 1, 3, 4, 66, 67, 68, 3 * 68 + 5, 1000])
def test_small_shapes_all_boundaries(D, max_ctas, S0):
    # n_sink + W = 68: S0 (+ gamma=3 appends) crosses empty, sink-only, window-fill, exactly-full and wrapped states
    _run_and_check(_cfg(S0=S0, D=D, W=64, n_sink=4, seed=100 + S0), max_ctas=max_ctas)


@pytest.mark.parametrize("D", [128, 256])
@pytest.mark.parametrize("max_ctas", [2, 4, 6, 8, 10, 14, 16, 22, 26, 32])
def test_windowed_cluster_sizes(D, max_ctas):
    # windowed launches run one thread-block cluster per (sequence, KV head); with two such pairs the CTA cap selects
    # clusters of 1, 2, 3, 4, 5, 7, 8, 11, 13 and 16 CTAs (any size up to 16 is used, not only powers of two). 1100 ring
    # slots are 18 tiles: ranks with one tile and ranks with two or three, output columns that do not divide evenly.
    _run_and_check(_cfg(S0=5000, D=D, W=1096, n_sink=4, gamma=3, seed=4100 + max_ctas), max_ctas=max_ctas)


@pytest.mark.parametrize("paged", [False, True])
@pytest.mark.parametrize("max_ctas", [3, 0])
def test_batched_ragged_lengths(paged, max_ctas):
    cfg = _cfg(batch=5, S0=0, S0_range=(1, 2000), paged=paged, W=128, n_sink=4, gamma=2, seed=77)
    _run_and_check(cfg, max_ctas=max_ctas)


@pytest.mark.parametrize("max_ctas", [1, 2, 0])
@pytest.mark.parametrize("D", [128, 256])
def test_many_short_sequences_one_cta_touches_many_segments(max_ctas, D):
    # 48 sequences x 2 KV heads = 96 segments: with one or two CTAs a consumer group contributes to more segments than
    # it can keep outstanding, so it has to combine part-way through its range
    cfg = _cfg(batch=48, S0=0, S0_range=(1, 400), D=D, W=64, n_sink=4, gamma=2, seed=4242)
    _run_and_check(cfg, max_ctas=max_ctas, check_ring=False)


def test_large_batch_of_short_sequences():
    cfg = _cfg(batch=300, S0=0, S0_range=(1, 150), D=128, W=32, n_sink=2, gamma=1, seed=99, paged=True)
    _run_and_check(cfg, check_ring=False, seqs=[0, 1, 57, 150, 298, 299])


def test_batch_with_empty_sequences():
    cfg = _cfg(batch=4, S0=0, S0_range=(1, 300), gamma=1, seed=5)
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    dw.lens[1] = 0; dw.lens[3] = 0          # two sequences hold no token
    out = torch.full((cfg.batch, cfg.Hq, cfg.D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((cfg.batch, cfg.Hq), float("nan"), device="cuda")
    wm.wmtp_draft_attn_full(dw.q[0], dw.kv, out, dw.ws, lse=lse)
    wm.wmtp_device_status(dw.ws)
    for b in (1, 3):
        assert (out[b] == 0).all() and torch.isneginf(lse[b]).all()
    for b in (0, 2):
        S = int(wl.seq_lens[b])
        ro, rl = R.attention(wl.q[0, b], np.ascontiguousarray(wl.K[b][:, :S]), np.ascontiguousarray(wl.V[b][:, :S]))
        compare(out[b], lse[b], ro, rl, what=f"seq {b}")


@pytest.mark.parametrize("cap_slack", [1, 6, 64])
@pytest.mark.parametrize("S0", [10, 70, 75, 140, 500])
def test_ring_with_slack_slots_reads_only_last_W(cap_slack, S0):
    _run_and_check(_cfg(S0=S0, W=64, n_sink=4, cap_slack=cap_slack, seed=300 + S0), max_ctas=0)
    _run_and_check(_cfg(S0=S0, W=64, n_sink=4, cap_slack=cap_slack, seed=300 + S0, D=256), max_ctas=5)


def test_windowed_equals_full_when_window_covers_context():
    cfg = _cfg(S0=200, W=256, n_sink=4, D=256)
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    dw.run_loops()
    # same keys, same values: both within tolerance of the oracle, and of each other
    d = (dw.out_w.float() - dw.out_f.float()).abs()
    assert d.max().item() <= 2e-2 and (dw.lse_w - dw.lse_f).abs().max().item() <= 1e-3
    _run_and_check(cfg)


# ------------------------------------------------------------------------------------------ structured inputs
@pytest.mark.parametrize("D", [128, 256])
def test_uniform_keys_give_mean_of_values(D):
    cfg = _cfg(S0=1500, D=D, W=256, gamma=1, seed=8)
    wl = wi.make_workload(cfg)
    wl.K_dev[:, :, :, :] = wl.K_dev[:, :, :1, :]          # every key row identical (views in wl.K follow)
    wl.k_new[:] = wl.K_dev[0, :, 0][None, None]
    Vf = wi.bf16_bits_to_f32(wl.V_dev) + 1.0               # V with mean 1: O(1) outputs
    wl.V_dev[...] = wi.f32_to_bf16_bits(Vf)
    dw = DeviceWorkload(wl)
    dw.run_loops()
    orc = oracle_for(wl, 0)
    r = orc.step(wl.q[0, 0], wl.k_new[0, 0], wl.v_new[0, 0])
    compare(dw.out_w[0, 0], dw.lse_w[0, 0], *r["win"], what="uniform windowed")
    compare(dw.out_f[0, 0], dw.lse_f[0, 0], *r["full"], what="uniform full")
    # closed form, independent of the oracle: mean of V over the key set
    S = orc.S
    meanV = wi.bf16_bits_to_f64(orc.Vfull[:, :S]).mean(axis=1)
    got = dw.out_f[0, 0].float().cpu().numpy().reshape(cfg.Hkv, cfg.G, D)
    assert np.abs(got - meanV[:, None, :]).max() <= 8e-3 * np.abs(meanV).max() + 1e-3


def test_planted_needle_full_finds_it_windowed_does_not():
    cfg = _cfg(S0=5000, D=128, W=256, gamma=1, seed=21)
    wl = wi.make_workload(cfg)
    qf = wi.bf16_bits_to_f32(wl.q[0, 0, 0])
    wl.K_dev[0, 0, 1234] = wi.f32_to_bf16_bits(qf * 2.0)     # logit ~ 2*|q|^2/sqrt(D) ~ 22 above the bulk
    dw = DeviceWorkload(wl)
    dw.run_loops()
    orc = oracle_for(wl, 0)
    r = orc.step(wl.q[0, 0], wl.k_new[0, 0], wl.v_new[0, 0])
    compare(dw.out_w[0, 0], dw.lse_w[0, 0], *r["win"], what="needle windowed")
    compare(dw.out_f[0, 0], dw.lse_f[0, 0], *r["full"], what="needle full")
    needle_v = wi.bf16_bits_to_f64(wl.V_dev[0, 0, 1234])
    got_f = dw.out_f[0, 0, 0].float().cpu().numpy()
    got_w = dw.out_w[0, 0, 0].float().cpu().numpy()
    assert np.abs(got_f - needle_v).max() < 0.05 and np.abs(got_w - needle_v).max() > 0.5
    mass = math.exp(float(dw.lse_w[0, 0, 0]) - float(dw.lse_f[0, 0, 0]))
    assert mass < 1e-3


def test_attention_mass_diagnostics_match_oracle():
    cfg = _cfg(S0=3000, D=128, W=256, gamma=2, seed=33, key_scale=(1.5, 2.5))     # peaked softmax: O(0.1..1) read-outs
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    dw.run_loops()
    rows = cfg.gamma * cfg.Hq
    mass, perturb, tail = (torch.full((rows,), float("nan"), device="cuda") for _ in range(3))
    wm.wmtp_attn_mass_diagnostics(dw.out_w, dw.lse_w, dw.out_f, dw.lse_f, mass=mass, perturb=perturb, tail=tail)
    orc = oracle_for(wl, 0)
    for i in range(cfg.gamma):
        r = orc.step(wl.q[i, 0], wl.k_new[i, 0], wl.v_new[i, 0])
        (ow, lw), (of, lf) = r["win"], r["full"]
        sl = slice(i * cfg.Hq, (i + 1) * cfg.Hq)
        np.testing.assert_allclose(mass[sl].cpu().numpy(), R.in_window_mass(lw, lf), rtol=2e-3, atol=1e-6)
        # the device works from the bf16 outputs: allow their rounding (2^-9 relative per element on both vectors)
        np.testing.assert_allclose(perturb[sl].cpu().numpy(), R.win_perturb(of, ow), atol=1e-2, rtol=1e-2)
        np.testing.assert_allclose(tail[sl].cpu().numpy(), R.tail_out_frac(of, ow, lw, lf), atol=1e-2, rtol=1e-2)
    m = mass.cpu().numpy()
    assert ((m > 0) & (m <= 1 + 1e-6)).all()


@pytest.mark.parametrize("target", [0.78, 0.16])
def test_attention_mass_on_structured_logit_profiles(target):
    """Recency-peaked logits calibrated to the in-window mass of a locally peaked (RoPE-like, ~0.75-0.80) and of a
    diffuse (NoPE-like, 0.16) head of the attention-mass table (Appendix D): the device diagnostics reproduce the
    oracle's figures, and both land on the calibration target."""
    S0, W, n_sink, tau = 200000, 4096, 4, 2048.0
    delta = wi.calibrate_delta(S0 + 1, n_sink, W, tau, target)
    cfg = _cfg(S0=S0, D=256, W=W, n_sink=n_sink, gamma=1, seed=61, logit_profile=(delta, tau), name=f"profile{target}")
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    dw.run_loops()
    mass, perturb, tail = (torch.full((cfg.Hq,), float("nan"), device="cuda") for _ in range(3))
    wm.wmtp_attn_mass_diagnostics(dw.out_w[0], dw.lse_w[0], dw.out_f[0], dw.lse_f[0], mass=mass, perturb=perturb, tail=tail)
    orc = oracle_for(wl, 0, with_ring=False)
    r = orc.step(wl.q[0, 0], wl.k_new[0, 0], wl.v_new[0, 0])
    (ow, lw), (of, lf) = r["win"], r["full"]
    compare(dw.out_w[0, 0], dw.lse_w[0, 0], ow, lw, what="profile windowed")
    compare(dw.out_f[0, 0], dw.lse_f[0, 0], of, lf, what="profile full")
    ref_mass = R.in_window_mass(lw, lf)
    np.testing.assert_allclose(mass.cpu().numpy(), ref_mass, rtol=2e-3, atol=1e-6)
    np.testing.assert_allclose(perturb.cpu().numpy(), R.win_perturb(of, ow), atol=2e-2, rtol=2e-2)
    np.testing.assert_allclose(tail.cpu().numpy(), R.tail_out_frac(of, ow, lw, lf), atol=2e-2, rtol=2e-2)
    assert abs(float(ref_mass.mean()) - target) < 0.06          # the noise of the other 255 dimensions averages out
    # far keys carry (1 - mass) of the weight: dropping them moves the read-out more for the diffuse profile
    assert (float(perturb.mean()) > 0.5) == (target < 0.5)


def test_explicit_softmax_scale():
    cfg = _cfg(S0=700, D=128, gamma=1)
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    out = torch.empty((1, cfg.Hq, cfg.D), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((1, cfg.Hq), device="cuda")
    wm.wmtp_draft_attn_full(dw.q[0], dw.kv, out, dw.ws, lse=lse, sm_scale=0.25)
    ro, rl = R.attention(wl.q[0, 0], np.ascontiguousarray(wl.K[0]), np.ascontiguousarray(wl.V[0]), sm_scale=0.25)
    compare(out[0], lse[0], ro, rl, what="scale 0.25")


def test_draft_loops_replay_from_a_cuda_graph():
    # lengths live on the device and are advanced by the kernels, so a captured loop can be replayed as is
    cfg = _cfg(S0=3000, D=256, W=256, gamma=3, seed=61)
    wl = wi.make_workload(cfg, extra_cap=16)
    dw = DeviceWorkload(wl)
    wm.wmtp_ring_init_from_kv(dw.ring, dw.kv)
    torch.cuda.synchronize()
    g, s = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            wm.wmtp_draft_loop_windowed(dw.ring, dw.q, dw.k_new, dw.v_new, dw.out_w, dw.ws, lse=dw.lse_w)
            wm.wmtp_draft_loop_full(dw.kv, dw.q, dw.k_new, dw.v_new, dw.out_f, dw.ws, lse=dw.lse_f)
    orc = oracle_for(wl, 0)
    orc_reserve = orc.Kfull.shape[1]
    assert orc_reserve >= cfg.S0 + 2 * cfg.gamma
    for replay in range(2):
        g.replay()
        torch.cuda.synchronize()
        wm.wmtp_device_status(dw.ws)
        for i in range(cfg.gamma):
            r = orc.step(wl.q[i, 0], wl.k_new[i, 0], wl.v_new[i, 0])
            compare(dw.out_w[i, 0], dw.lse_w[i, 0], *r["win"], what=f"graph replay {replay} step {i} windowed")
            compare(dw.out_f[i, 0], dw.lse_f[i, 0], *r["full"], what=f"graph replay {replay} step {i} full")
        assert int(dw.lens[0]) == orc.S and int(dw.ring.len[0]) == orc.S
    check_ring_against_sim(dw.ring, 0, orc.ring, "after two graph replays")


def test_host_buffer_loop_matches_device_loop():
    cfg = _cfg(S0=900, D=256, W=128, gamma=3)
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    dw.run_loops()
    dw2 = DeviceWorkload(wl)
    stage = torch.empty(wm.wmtp_stage_bytes(cfg.gamma, 1, cfg.Hq, cfg.Hkv, cfg.D), dtype=torch.uint8, device="cuda")
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).pin_memory()
    qh, kh, vh = pin(wl.q), pin(wl.k_new), pin(wl.v_new)
    oh_w, oh_f = torch.empty_like(qh).pin_memory(), torch.empty_like(qh).pin_memory()
    lh = torch.empty(qh.shape[:-1], dtype=torch.float32).pin_memory()
    wm.wmtp_ring_init_from_kv(dw2.ring, dw2.kv)
    wm.wmtp_draft_loop_windowed_host(dw2.ring, qh, kh, vh, oh_w, stage, dw2.ws, lse_host=lh)
    # same kernels on the same bits; equal up to the order in which split-KV partials are summed
    assert (oh_w.float() - dw.out_w.cpu().float()).abs().max().item() <= 4e-3
    assert (lh - dw.lse_w.cpu()).abs().max().item() <= 1e-4
    wm.wmtp_draft_loop_full_host(dw2.kv, qh, kh, vh, oh_f, stage, dw2.ws)
    assert (oh_f.float() - dw.out_f.cpu().float()).abs().max().item() <= 4e-3


# ------------------------------------------------------------------------------------------ benchmark configurations
def test_config_tiny_full_gamma_loop():
    _run_and_check(wi.CONFIGS[0])


def test_fixed_partition_is_bit_reproducible_and_stealing_agrees():
    cfg = wi.scaled(wi.CONFIGS[1], S0=40000, gamma=2, name="repro")
    wl = wi.make_workload(cfg)
    outs = []
    for stealing in (False, False, True):
        wm.wmtp_set_work_stealing(stealing)
        dw = DeviceWorkload(wl)
        dw.run_loops()
        outs.append((dw.out_f.clone(), dw.lse_f.clone(), dw.out_w.clone()))
    assert torch.equal(outs[0][0].view(torch.int16), outs[1][0].view(torch.int16))
    assert torch.equal(outs[0][1], outs[1][1]) and torch.equal(outs[0][2].view(torch.int16), outs[1][2].view(torch.int16))
    assert (outs[0][0].float() - outs[2][0].float()).abs().max().item() <= 4e-3
    assert (outs[0][1] - outs[2][1]).abs().max().item() <= 1e-4


def test_config_s128k():
    _run_and_check(wi.CONFIGS[1])


def test_config_million_token_all_heads():
    # full size, in the launch configuration the benchmark times (default CTAs); first and last draft step
    _run_and_check(wi.CONFIGS[2], steps={0, 6})


def test_config_batched_paged_reduced_and_full_size_sample():
    small = wi.scaled(wi.CONFIGS[3], batch=6, S0_range=(2048, 65536), gamma=3, name="batched_small")
    _run_and_check(small)


def test_config_batched_paged_full_size_sampled_sequences():
    cfg = wi.scaled(wi.CONFIGS[3], gamma=2, name="batched_full")
    lens = wi.seq_lens(cfg)
    order = np.argsort(lens)
    sample = [int(order[0]), int(order[len(order) // 2]), int(order[-1])]      # shortest, median, longest
    _run_and_check(cfg, seqs=sample, check_ring=True)


@pytest.mark.parametrize("S0,W", [(65536, 1024), (262144, 4096)])
def test_config_sweep_shapes(S0, W):
    _run_and_check(wi.scaled(wi.CONFIGS[4], S0=S0, W=W, gamma=3, name=f"sweep_{S0}_{W}"))


def test_config_sweep_shape_at_full_size():
    # Hq=32, Hkv=4, D=128 at S=1,048,576 (the two-consumer-group kernel at the size the benchmark times), default CTAs;
    # first and last draft step
    _run_and_check(wi.scaled(wi.CONFIGS[4], name="sweep_full_size"), steps={0, 6})


def test_two_host_threads_on_their_own_streams_and_workspaces():
    """Two host threads drive their own stores, workspaces and streams at the same time (the library's per-device caches
    are shared between them; cooperative launches of the two streams take the GPU in turn): both must match the oracle."""
    import threading

    cfgs = [wi.DraftConfig("thrA", 1, 3000, 16, 2, 256, 256, 4, 3, seed=91),
            wi.DraftConfig("thrB", 2, 0, 8, 2, 128, 64, 4, 3, seed=92, S0_range=(500, 5000), paged=True)]
    wls = [wi.make_workload(c) for c in cfgs]
    dws = [DeviceWorkload(w) for w in wls]
    streams = [torch.cuda.Stream() for _ in cfgs]
    errors = []

    def run(i):
        try:
            dw, st = dws[i], streams[i]
            with torch.cuda.stream(st):
                for _ in range(3):                                   # the same loops three times over: lengths restored in between
                    dw.lens.copy_(torch.from_numpy(wls[i].seq_lens.copy()), non_blocking=False)
                    wm.wmtp_ring_init_from_kv(dw.ring, dw.kv, stream=st.cuda_stream)
                    wm.wmtp_draft_loop_windowed(dw.ring, dw.q, dw.k_new, dw.v_new, dw.out_w, dw.ws, lse=dw.lse_w, stream=st.cuda_stream)
                    wm.wmtp_draft_loop_full(dw.kv, dw.q, dw.k_new, dw.v_new, dw.out_f, dw.ws, lse=dw.lse_f, stream=st.cuda_stream)
                wm.wmtp_device_status(dw.ws, stream=st.cuda_stream)
        except Exception as exc:                                     # surfaces in the main thread below
            errors.append(exc)

    threads = [threading.Thread(target=run, args=(i,)) for i in range(len(cfgs))]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert not errors, errors
    for i, (cfg, wl, dw) in enumerate(zip(cfgs, wls, dws)):
        dw.guard.check(cfg.name)
        for b in range(cfg.batch):
            orc = oracle_for(wl, b)
            for s in range(cfg.gamma):
                r = orc.step(wl.q[s, b], wl.k_new[s, b], wl.v_new[s, b])
                compare(dw.out_w[s, b], dw.lse_w[s, b], *r["win"], what=f"{cfg.name} seq={b} step={s} windowed")
                compare(dw.out_f[s, b], dw.lse_f[s, b], *r["full"], what=f"{cfg.name} seq={b} step={s} full")
