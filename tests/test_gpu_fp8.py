"""GPU parity of the fp8 (e4m3) KV variant: stores hold one-byte codes with a scale per KV head, new rows are
quantised on append (bit-exact against the oracle's quantiser), attention dequantises exactly."""
import numpy as np
import pytest
import torch

import paper_2607_21535_b200 as wm
import wmtp_inputs as wi
from oracle import reference as R

from harness import DeviceWorkload, bits, check_ring_against_sim, compare, oracle_for, to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _defaults():
    wm.wmtp_set_max_ctas(0)
    wm.wmtp_set_work_stealing(True)
    yield
    wm.wmtp_set_max_ctas(0)
    wm.wmtp_set_work_stealing(True)


def _cfg(**kw):
    base = dict(name="f8", batch=1, S0=300, Hq=16, Hkv=2, D=128, W=64, n_sink=4, gamma=3, seed=8800, kv_dtype="fp8",
                key_scale=(0.5, 2.0))
    base.update(kw)
    return wi.DraftConfig(**base)


def _per_seq(a):
    return np.ascontiguousarray(np.swapaxes(a, 0, 1))


# ------------------------------------------------------------------------------------------ store operations
@pytest.mark.parametrize("D", [128, 256])
def test_ring_append_quantises_bit_exactly(D):
    """Rows of every magnitude: far below the smallest code, subnormal codes, the normal range, beyond 448 scales
    (saturation), exact ties between codes, zeros of both signs."""
    B, Hkv, n_sink, W, cap = 2, 2, 4, 8, 11
    n = 3 * (n_sink + cap) + 5
    rs = np.random.RandomState(D)
    mag = np.exp(rs.uniform(np.log(1e-6), np.log(50.0), (n, B, Hkv, 1))).astype(np.float32)
    kf = wi.bf16_bits_to_f32(wi.normal_bf16(12, (1, D), (n, B, Hkv, D))) * mag
    vf = wi.bf16_bits_to_f32(wi.normal_bf16(12, (2, D), (n, B, Hkv, D))) * mag
    k_scale, v_scale = np.float32([0.0123, 0.5]), np.float32([1.0, 0.031])
    table = R.e4m3_decode(np.arange(0x7F, dtype=np.uint8))
    ties = ((table[:-1] + table[1:]) / 2).astype(np.float32)                       # ties in units of the scale ...
    kf[0, 0, 1, :ties.size] = ties[:D]                                             # ... exact for the head whose scale is 0.5
    kf[0, 0, 1, :ties.size] *= 0.5
    vf[0, 0, 0, :ties.size] = -ties[:D]                                            # head with scale 1.0
    kf[1, 0, 0, :4] = [0.0, -0.0, 1e30, -1e30]
    k, v = wi.f32_to_bf16_bits(kf), wi.f32_to_bf16_bits(vf)
    kd, vd = to_dev_bf16(k), to_dev_bf16(v)
    ks, vs = torch.from_numpy(k_scale).cuda(), torch.from_numpy(v_scale).cuda()
    ring = wm.Ring(B, Hkv, D, n_sink, W, cap=cap, k_scale=ks, v_scale=vs)
    ring.k.fill_(0x7F); ring.v.fill_(0x7F)
    wm.wmtp_ring_reset(ring)
    sims = [R.RingSim(n_sink, cap, Hkv, D, dtype=np.uint8) for _ in range(B)]
    for i in range(n):
        wm.wmtp_ring_append(ring, kd[i], vd[i])
        for b in range(B):
            sims[b].append(R.quantize_rows(k[i, b], k_scale), R.quantize_rows(v[i, b], v_scale))
    for b in range(B):
        check_ring_against_sim(ring, b, sims[b], f"fp8 ring seq {b}")
    codes = bits(ring.k)
    assert not ((codes & 0x7F) == 0x7F).any()                                      # saturation, never a NaN code


@pytest.mark.parametrize("paged", [False, True])
def test_kv_append_many_and_single_quantise_identically(paged):
    cfg = _cfg(batch=3, S0=0, S0_range=(40, 300), paged=paged, gamma=5, cap_slack=5)
    wl = wi.make_workload(cfg)
    a, b_ = DeviceWorkload(wl), DeviceWorkload(wl)
    for dw in (a, b_):
        wm.wmtp_ring_init_from_kv(dw.ring, dw.kv)
    for i in range(cfg.gamma):
        wm.wmtp_ring_append(a.ring, a.k_new[i], a.v_new[i])
        wm.wmtp_kv_append(a.kv, a.k_new[i], a.v_new[i], a.ws)
    km, vm = to_dev_bf16(_per_seq(wl.k_new)), to_dev_bf16(_per_seq(wl.v_new))
    wm.wmtp_ring_append_many(b_.ring, km, vm)
    wm.wmtp_kv_append_many(b_.kv, km, vm, b_.ws)
    wm.wmtp_device_status(a.ws); wm.wmtp_device_status(b_.ws)
    for x, y in ((a.ring.k, b_.ring.k), (a.ring.v, b_.ring.v), (a.K, b_.K), (a.V, b_.V)):
        assert (bits(x) == bits(y)).all()
    for b in range(cfg.batch):
        orc = oracle_for(wl, b)
        for i in range(cfg.gamma):
            orc.append(wl.k_new[i, b], wl.v_new[i, b])
        check_ring_against_sim(a.ring, b, orc.ring, f"seq {b}")
        S = orc.S
        if not paged:
            assert (bits(a.K[b])[:, :S] == orc.Kfull[:, :S]).all() and (bits(a.V[b])[:, :S] == orc.Vfull[:, :S]).all()


def test_ring_init_rejects_mixed_dtypes():
    wl8, wl16 = wi.make_workload(_cfg()), wi.make_workload(_cfg(kv_dtype="bf16"))
    d8, d16 = DeviceWorkload(wl8), DeviceWorkload(wl16)
    with pytest.raises(wm.WmtpError) as ei:
        wm.wmtp_ring_init_from_kv(d8.ring, d16.kv)
    assert ei.value.status == 1


# ------------------------------------------------------------------------------------------ attention parity
def _run_and_check(cfg, max_ctas=0, seqs=None, steps=None, check_store=True):
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    wm.wmtp_set_max_ctas(max_ctas)
    dw.run_loops()
    for b in (range(cfg.batch) if seqs is None else seqs):
        orc = oracle_for(wl, b, with_ring=check_store)
        for i in range(cfg.gamma):
            do = steps is None or i in steps
            r = orc.step(wl.q[i, b], wl.k_new[i, b], wl.v_new[i, b], full=do, windowed=do)
            if do:
                tag = f"{cfg.name} ctas={max_ctas} seq={b} step={i}"
                compare(dw.out_w[i, b], dw.lse_w[i, b], *r["win"], what=tag + " windowed")
                compare(dw.out_f[i, b], dw.lse_f[i, b], *r["full"], what=tag + " full")
        if check_store:
            check_ring_against_sim(dw.ring, b, orc.ring, f"{cfg.name} seq={b}")     # the fused appends quantised the same codes
            if not cfg.paged:
                S0, S = int(wl.seq_lens[b]), orc.S
                assert (bits(dw.K[b])[:, S0:S] == orc.Kfull[:, S0:S]).all() and (bits(dw.V[b])[:, S0:S] == orc.Vfull[:, S0:S]).all()
        assert int(dw.lens[b]) == orc.S


@pytest.mark.parametrize("D", [128, 256])
@pytest.mark.parametrize("max_ctas", [1, 2, 7, 0])
@pytest.mark.parametrize("S0", [0, 1, 3, 4, 66, 67, 68, 3 * 68 + 5, 1000])
def test_small_shapes_all_boundaries(D, max_ctas, S0):
    _run_and_check(_cfg(S0=S0, D=D, seed=100 + S0), max_ctas=max_ctas)


@pytest.mark.parametrize("paged", [False, True])
@pytest.mark.parametrize("D", [128, 256])
def test_batched_ragged_lengths(paged, D):
    _run_and_check(_cfg(batch=5, S0=0, S0_range=(1, 3000), paged=paged, D=D, W=128, gamma=2, seed=77))


@pytest.mark.parametrize("max_ctas", [1, 3, 0])
@pytest.mark.parametrize("S0", [62, 63, 64, 126, 127, 128, 190, 191, 192, 320])
def test_paired_tiles_odd_and_even_tile_counts(S0, max_ctas):
    """head_dim 128 fp8 stores travel two tiles to a stage: lengths around tile boundaries give stages of one and of
    two tiles, and put the appended row into the first and into the second tile of a pair (gamma = 3 appends)."""
    _run_and_check(_cfg(S0=S0, D=128, seed=500 + S0), max_ctas=max_ctas)


@pytest.mark.parametrize("paged", [False, True])
@pytest.mark.parametrize("stealing", [True, False])
def test_paired_tiles_long_ragged_batch(paged, stealing):
    """Ranges long enough for the cursor-driven tail (and thieves) on a ragged batch (37 CTAs over some 9000 tiles):
    chunks and stolen runs end at segment ends, where a stage may hold a single tile."""
    wm.wmtp_set_work_stealing(stealing)
    _run_and_check(_cfg(batch=3, S0=0, S0_range=(150001, 260000), paged=paged, D=128, Hq=8, Hkv=1, W=512, gamma=2, seed=91),
                   max_ctas=37, check_store=False)


@pytest.mark.parametrize("Hq,Hkv", [(8, 8), (4, 2), (32, 4), (6, 2)])
def test_group_sizes(Hq, Hkv):
    _run_and_check(_cfg(Hq=Hq, Hkv=Hkv, S0=900, key_scale=None, seed=Hq * 10 + Hkv), max_ctas=0)


def test_ring_with_slack_slots():
    for S0 in (10, 75, 500):
        _run_and_check(_cfg(S0=S0, cap_slack=6, seed=300 + S0, D=256))


def test_query_scale_extremes():
    """The query is normalised by a power of two per head before the f16 MMA: huge and tiny queries keep their result."""
    cfg = _cfg(S0=700, D=256, gamma=1, seed=5150)
    wl = wi.make_workload(cfg)
    qf = wi.bf16_bits_to_f32(wl.q)
    qf[0, 0, :4] *= 2.0 ** 20         # far beyond the f16 range
    qf[0, 0, 4:8] *= 2.0 ** -30       # far below f16's smallest normal
    qf[0, 0, 8] = 0.0
    wl.q = wi.f32_to_bf16_bits(qf)
    dw = DeviceWorkload(wl)
    dw.run_loops()
    orc = oracle_for(wl, 0)
    # a softmax scale that keeps the logits of the huge heads finite and non-degenerate
    r = orc.step(wl.q[0, 0], wl.k_new[0, 0], wl.v_new[0, 0])
    out_f = dw.out_f[0, 0].float().cpu().numpy()
    assert np.isfinite(out_f).all()
    for h in list(range(4, 16)):       # moderate, tiny and zero heads: ordinary tolerance
        compare(dw.out_f[0, 0][h:h + 1], dw.lse_f[0, 0][h:h + 1], r["full"][0][h:h + 1], r["full"][1][h:h + 1], what=f"head {h}")
    # huge heads: the softmax is a near one-hot; the winner must be the oracle's winner
    for h in range(4):
        assert np.abs(out_f[h] - r["full"][0][h]).max() <= 2e-2 * max(1.0, np.abs(r["full"][0][h]).max())


def test_windowed_kv_view_and_extend_on_fp8_store():
    cfg = _cfg(S0=1500, D=256, W=128, gamma=4, cap_slack=4, seed=909)
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    ws = wm.Workspace(cfg.batch * cfg.gamma, cfg.Hq, cfg.Hkv, cfg.D)
    wm.wmtp_ring_init_from_kv(dw.ring, dw.kv)
    km, vm, qm = to_dev_bf16(_per_seq(wl.k_new)), to_dev_bf16(_per_seq(wl.v_new)), to_dev_bf16(_per_seq(wl.q))
    wm.wmtp_ring_append_many(dw.ring, km, vm)
    wm.wmtp_kv_append_many(dw.kv, km, vm, ws)
    out_w, out_f = torch.empty_like(qm), torch.empty_like(qm)
    lse_w = torch.empty(qm.shape[:-1], dtype=torch.float32, device="cuda")
    lse_f = torch.empty_like(lse_w)
    wm.wmtp_draft_extend_windowed(qm, dw.ring, out_w, ws, lse=lse_w)
    wm.wmtp_draft_extend_full(qm, dw.kv, out_f, ws, lse=lse_f)
    out_v = torch.empty_like(dw.q[0]); lse_v = torch.empty_like(dw.lse_w[0])
    wm.wmtp_draft_attn_windowed_kv(qm[:, -1].contiguous(), dw.kv, cfg.n_sink, cfg.W, out_v, dw.ws, lse=lse_v)
    wm.wmtp_device_status(ws); wm.wmtp_device_status(dw.ws)
    orc = oracle_for(wl, 0, with_ring=False)
    for i in range(cfg.gamma):
        r = orc.step(wl.q[i, 0], wl.k_new[i, 0], wl.v_new[i, 0])
        compare(out_w[0, i], lse_w[0, i], *r["win"], what=f"extend windowed token {i}")
        compare(out_f[0, i], lse_f[0, i], *r["full"], what=f"extend full token {i}")
    compare(out_v[0], lse_v[0], *r["win"], what="window view over the fp8 KV store")


def test_fixed_partition_is_bit_reproducible():
    cfg = _cfg(S0=40000, D=256, W=2048, gamma=2, seed=1235, name="f8repro")
    wl = wi.make_workload(cfg)
    outs = []
    for _ in range(2):
        wm.wmtp_set_work_stealing(False)
        dw = DeviceWorkload(wl)
        dw.run_loops()
        outs.append((dw.out_f.clone(), dw.lse_f.clone(), dw.out_w.clone()))
    assert torch.equal(outs[0][0].view(torch.int16), outs[1][0].view(torch.int16))
    assert torch.equal(outs[0][1], outs[1][1]) and torch.equal(outs[0][2].view(torch.int16), outs[1][2].view(torch.int16))


# ------------------------------------------------------------------------------------------ benchmark shapes
def test_config_s128k_fp8():
    _run_and_check(wi.scaled(wi.CONFIGS[1], kv_dtype="fp8", name="s128k_fp8"))


def test_config_million_token_fp8():
    _run_and_check(wi.scaled(wi.CONFIGS[2], kv_dtype="fp8", name="million_fp8"), steps={0, 6})


def test_config_batched_paged_fp8_reduced():
    _run_and_check(wi.scaled(wi.CONFIGS[3], batch=6, S0_range=(2048, 65536), gamma=3, kv_dtype="fp8", name="batched_fp8"))


def test_config_sweep_shape_fp8():
    _run_and_check(wi.scaled(wi.CONFIGS[4], S0=262144, W=4096, gamma=3, kv_dtype="fp8", name="sweep_fp8"))


def test_config_sweep_shape_fp8_at_full_size():
    """The head_dim-128 shape at the size the benchmark times it (S = 1,048,576; tiles in pairs), first and last step."""
    _run_and_check(wi.scaled(wi.CONFIGS[4], kv_dtype="fp8", name="sweep_fp8_full_size"), steps={0, 6})


@pytest.mark.parametrize("kv_dtype,D", [("fp8", 256), ("fp8", 128), ("bf16", 128), ("bf16", 256)])
def test_very_large_batch_leaves_room_for_fewer_stages(kv_dtype, D):
    """1000 sequences: the batch-sized tables take shared memory from the stage ring, the kernel runs with fewer stages."""
    cfg = _cfg(batch=1000, S0=0, S0_range=(1, 200), D=D, W=32, n_sink=2, gamma=1, seed=4711, paged=True, kv_dtype=kv_dtype,
               key_scale=None)
    _run_and_check(cfg, seqs=[0, 1, 333, 500, 998, 999], check_store=False)
