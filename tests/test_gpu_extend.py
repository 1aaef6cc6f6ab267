"""Rollback of rejected tokens and draft-extend (several new tokens per sequence in one launch), against the oracle's
sequential decode steps and its slot-level ring simulation."""
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


def _cfg(**kw):
    base = dict(name="ext", batch=1, S0=300, Hq=16, Hkv=2, D=128, W=64, n_sink=4, gamma=5, seed=808)
    base.update(kw)
    return wi.DraftConfig(**base)


def _per_seq(a):
    """[gamma][B][...] -> contiguous [B][gamma][...] (the layout of the *_many / extend calls)."""
    return np.ascontiguousarray(np.swapaxes(a, 0, 1))


# ------------------------------------------------------------------------------------------ store operations
@pytest.mark.parametrize("n_sink,W,slack", [(4, 8, 3), (0, 5, 7), (2, 16, 16)])
def test_ring_rewind_then_append_bit_exact(n_sink, W, slack):
    B, Hkv, D, cap = 2, 2, 128, W + slack
    n = 4 * (n_sink + cap)
    k = wi.normal_bf16(5, (1, n_sink, W), (n, B, Hkv, D))
    v = wi.normal_bf16(5, (2, n_sink, W), (n, B, Hkv, D))
    kd, vd = to_dev_bf16(k), to_dev_bf16(v)
    ring = wm.Ring(B, Hkv, D, n_sink, W, cap=cap)
    wm.wmtp_ring_reset(ring)
    sims = [R.RingSim(n_sink, cap, Hkv, D) for _ in range(B)]
    rng = np.random.RandomState(n_sink + W)
    i = 0
    while i < n - (slack + 2):
        burst = int(rng.randint(1, slack + 2))
        for _ in range(burst):
            wm.wmtp_ring_append(ring, kd[i], vd[i])
            for b in range(B):
                sims[b].append(k[i, b], v[i, b])
            i += 1
        drops = np.array([int(rng.randint(0, min(burst, slack) + 1)) for _ in range(B)], dtype=np.int32)
        wm.wmtp_ring_rewind(ring, torch.from_numpy(drops).cuda())
        for b in range(B):
            sims[b].rewind(int(drops[b]))
            check_ring_against_sim(ring, b, sims[b], f"after rewind at {i}")
        # the sequences now differ in length: re-align them so that one append call serves both
        catch_up = int(drops.max())
        for b in range(B):
            for _ in range(catch_up - int(drops[b])):
                sims[b].rewind(1)
        wm.wmtp_ring_rewind(ring, torch.from_numpy((catch_up - drops).astype(np.int32)).cuda())
        i -= catch_up
        assert all(s.length == i for s in sims)


def test_ring_rewind_beyond_slack_is_flagged_and_ignored():
    ring = wm.Ring(1, 2, 128, 4, 8, cap=10)
    ws = wm.Workspace(1, 16, 2, 128)
    wm.wmtp_ring_reset(ring)
    k = to_dev_bf16(wi.normal_bf16(1, 1, (20, 1, 2, 128)))
    for i in range(20):
        wm.wmtp_ring_append(ring, k[i], k[i])
    before = ring.slot_pos.clone()
    wm.wmtp_ring_rewind(ring, torch.tensor([3], dtype=torch.int32, device="cuda"), ws)      # slack is 2
    with pytest.raises(wm.WmtpError) as ei:
        wm.wmtp_device_status(ws)
    assert ei.value.status == 7 and int(ring.len[0]) == 20 and torch.equal(ring.slot_pos, before)


@pytest.mark.parametrize("kv_dtype", ["bf16", "fp8"])
def test_ring_replace_tail_equals_rewind_then_append(kv_dtype):
    """The one-launch state update after a verify step against the slot simulation: every (rejected, accepted) pair
    that fits the slack, including more rejected than accepted (left-over slots become empty) and none rejected."""
    B, Hkv, D, n_sink, W, slack = 3, 2, 128, 4, 16, 6
    cap = W + slack
    f8 = kv_dtype == "fp8"
    k_scale, v_scale = np.float32([0.02, 0.011]), np.float32([0.015, 0.03])
    ks = dict(k_scale=torch.from_numpy(k_scale).cuda(), v_scale=torch.from_numpy(v_scale).cuda()) if f8 else {}
    ring = wm.Ring(B, Hkv, D, n_sink, W, cap=cap, **ks)
    ws = wm.Workspace(B, 16, Hkv, D)
    wm.wmtp_ring_reset(ring)
    sims = [R.RingSim(n_sink, cap, Hkv, D, dtype=np.uint8 if f8 else np.uint16) for _ in range(B)]
    stored = (lambda rows, sc: R.quantize_rows(rows, sc)) if f8 else (lambda rows, sc: rows)
    rng = np.random.RandomState(17)
    tid = 0
    for it in range(40):
        n_tok = int(rng.randint(1, 8))
        drops = np.array([int(rng.randint(0, slack + 1)) for _ in range(B)], dtype=np.int32)
        drops = np.minimum(drops, [s.length for s in sims]).astype(np.int32)
        if it % 7 == 0:
            drops[:] = 0
        k = wi.normal_bf16(3, (1, it), (B, n_tok, Hkv, D)); v = wi.normal_bf16(3, (2, it), (B, n_tok, Hkv, D))
        wm.wmtp_ring_replace_tail(ring, torch.from_numpy(drops).cuda() if it % 7 else None, to_dev_bf16(k), to_dev_bf16(v), ws)
        for b in range(B):
            sims[b].rewind(int(drops[b]))
            for j in range(n_tok):
                sims[b].append(stored(k[b, j], k_scale), stored(v[b, j], v_scale))
            check_ring_against_sim(ring, b, sims[b], f"iteration {it} seq {b}")
    wm.wmtp_device_status(ws)
    before = ring.slot_pos.clone()
    wm.wmtp_ring_replace_tail(ring, torch.full((B,), slack + 1, dtype=torch.int32, device="cuda"), to_dev_bf16(k), to_dev_bf16(v), ws)
    with pytest.raises(wm.WmtpError) as ei:
        wm.wmtp_device_status(ws)
    assert ei.value.status == 7 and torch.equal(ring.slot_pos, before)


@pytest.mark.parametrize("paged", [False, True])
def test_append_many_equals_sequential_appends(paged):
    cfg = _cfg(batch=3, S0=0, S0_range=(50, 400), paged=paged, gamma=6, cap_slack=6)
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
    assert torch.equal(a.ring.slot_pos, b_.ring.slot_pos) and torch.equal(a.ring.len, b_.ring.len) and torch.equal(a.lens, b_.lens)


# ------------------------------------------------------------------------------------------ draft-extend attention
def _extend_and_check(cfg, max_ctas=0, seqs=None):
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    wm.wmtp_set_max_ctas(max_ctas)
    qlen = cfg.gamma
    ws = wm.Workspace(cfg.batch * qlen, cfg.Hq, cfg.Hkv, cfg.D)
    wm.wmtp_ring_init_from_kv(dw.ring, dw.kv)
    km, vm, qm = to_dev_bf16(_per_seq(wl.k_new)), to_dev_bf16(_per_seq(wl.v_new)), to_dev_bf16(_per_seq(wl.q))
    wm.wmtp_ring_append_many(dw.ring, km, vm)
    wm.wmtp_kv_append_many(dw.kv, km, vm, ws)
    out_w, out_f = torch.full_like(qm, float("nan")), torch.full_like(qm, float("nan"))
    lse_w = torch.full(qm.shape[:-1], float("nan"), dtype=torch.float32, device="cuda")
    lse_f = torch.full_like(lse_w, float("nan"))
    wm.wmtp_draft_extend_windowed(qm, dw.ring, out_w, ws, lse=lse_w)
    wm.wmtp_draft_extend_full(qm, dw.kv, out_f, ws, lse=lse_f)
    wm.wmtp_device_status(ws)
    dw.guard.check(cfg.name)                 # appends and extends wrote nothing outside the stores
    for b in (range(cfg.batch) if seqs is None else seqs):
        orc = oracle_for(wl, b, with_ring=False)
        for i in range(qlen):
            r = orc.step(wl.q[i, b], wl.k_new[i, b], wl.v_new[i, b])
            tag = f"{cfg.name} ctas={max_ctas} seq={b} token={i}"
            compare(out_w[b, i], lse_w[b, i], *r["win"], what=tag + " extend windowed")
            compare(out_f[b, i], lse_f[b, i], *r["full"], what=tag + " extend full")


@pytest.mark.parametrize("kv_dtype", ["bf16", "fp8"])
@pytest.mark.parametrize("D", [128, 256])
@pytest.mark.parametrize("S0", [0, 2, 60, 66, 70, 300, 2000])
@pytest.mark.parametrize("max_ctas", [1, 0])
def test_extend_matches_sequential_steps(D, S0, max_ctas, kv_dtype):
    # n_sink + W = 68 and five new tokens: the queries straddle sink-filling, window-filling and sliding states
    _extend_and_check(_cfg(S0=S0, D=D, cap_slack=4, seed=900 + S0, kv_dtype=kv_dtype), max_ctas=max_ctas)


@pytest.mark.parametrize("kv_dtype", ["bf16", "fp8"])
@pytest.mark.parametrize("paged", [False, True])
def test_extend_batched_ragged(paged, kv_dtype):
    _extend_and_check(_cfg(batch=4, S0=0, S0_range=(10, 3000), paged=paged, gamma=7, cap_slack=8, W=128, seed=31, kv_dtype=kv_dtype,
                           key_scale=(0.5, 2.0) if kv_dtype == "fp8" else None))


@pytest.mark.parametrize("kv_dtype", ["bf16", "fp8"])
def test_extend_at_long_context(kv_dtype):
    _extend_and_check(wi.scaled(wi.CONFIGS[1], gamma=7, cap_slack=6, kv_dtype=kv_dtype, name="ext_s128k_" + kv_dtype))


@pytest.mark.parametrize("D", [128, 256])
def test_extend_fp8_group_sizes_and_query_chunks(D):
    """fp8 store, six new tokens (two passes: a chunk of four queries and one of two), three query heads per KV head
    (heads beyond the group read as zero in the MMA tile), distinct scales per KV head."""
    _extend_and_check(_cfg(S0=700, D=D, Hq=6, Hkv=2, gamma=6, cap_slack=8, W=128, seed=77, kv_dtype="fp8", key_scale=(0.5, 2.0)))


def test_extend_needs_slack_slots():
    cfg = _cfg(S0=200, gamma=3, cap_slack=1)             # 3 tokens need cap >= W + 2
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    ws = wm.Workspace(3, cfg.Hq, cfg.Hkv, cfg.D)
    qm = to_dev_bf16(_per_seq(wl.q))
    with pytest.raises(wm.WmtpError) as ei:
        wm.wmtp_draft_extend_windowed(qm, dw.ring, torch.empty_like(qm), ws)
    assert ei.value.status == 3


def test_speculative_cycle_draft_rewind_extend():
    """gamma speculative draft steps, the target accepts `a` of them plus its own bonus token, the draft rolls back
    and re-processes the accepted tokens: the ring ends up exactly as if only those tokens had ever been appended."""
    cfg = _cfg(S0=500, D=256, W=128, gamma=6, cap_slack=7, seed=77)
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    dw.run_loops(full=False)                              # 6 speculative tokens in the ring
    accepted = 2
    wm.wmtp_ring_rewind(dw.ring, torch.tensor([cfg.gamma - accepted], dtype=torch.int32, device="cuda"), dw.ws)
    # the target's verified tokens: the two accepted ones plus a bonus token with its own K/V
    bonus_k = wi.normal_bf16(cfg.seed, 91, (1, 1, cfg.Hkv, cfg.D))
    bonus_v = wi.normal_bf16(cfg.seed, 92, (1, 1, cfg.Hkv, cfg.D))
    bonus_q = wi.normal_bf16(cfg.seed, 93, (1, 1, cfg.Hq, cfg.D))
    wm.wmtp_ring_append_many(dw.ring, to_dev_bf16(bonus_k), to_dev_bf16(bonus_v))
    qd = to_dev_bf16(bonus_q)
    out = torch.empty_like(qd)
    lse = torch.empty(qd.shape[:-1], dtype=torch.float32, device="cuda")
    wm.wmtp_draft_extend_windowed(qd, dw.ring, out, dw.ws, lse=lse)
    wm.wmtp_device_status(dw.ws)
    orc = oracle_for(wl, 0)
    for i in range(accepted):
        orc.step(wl.q[i, 0], wl.k_new[i, 0], wl.v_new[i, 0], full=False)
    r = orc.step(bonus_q[0, 0], bonus_k[0, 0], bonus_v[0, 0], full=False)
    compare(out[0, 0], lse[0, 0], *r["win"], what="bonus token after rollback")
    assert int(dw.ring.len[0]) == orc.S
    # every position of the kept set sits in the slot the oracle's ring has it in, with the same bits; no slot
    # claims a position at or beyond the new length
    pos = dw.ring.slot_pos[0].cpu().numpy()
    keep = set(R.keep_set(orc.S, cfg.n_sink, cfg.W))
    Kb = bits(dw.ring.k[0])
    seen = 0
    for s, p in enumerate(orc.ring.slot_pos):
        if int(p) in keep:
            assert pos[s] == p and (Kb[:, s] == orc.ring.K[:, s]).all()
            seen += 1
    assert seen == len(keep) and (pos < orc.S).all()


# ------------------------------------------------------------------------------------------ one workspace, changing shapes
@pytest.mark.parametrize("D", [128, 256])
def test_one_workspace_serves_extend_and_decode_launches_in_turn(D):
    """The normal speculative cycle on ONE workspace: a draft-extend launch (q_len times the (sequence, KV head) pairs
    of a decode step), some decode steps, the next extend, ... The kernels keep two copies of their per-segment words
    and each launch prepares the other copy for the next one, whose segment count may be larger than its own: with an
    odd number of decode launches between two extends the second extend lands on the copy the first one used. Every
    output is compared with the oracle's sequential steps."""
    q_len = 4
    cycles = [(3, False), (1, True), (2, False), (3, True)]      # (decode steps, also run the full-context loop)
    total = sum(q_len + d for d, _ in cycles)
    cfg = _cfg(batch=2, S0=0, S0_range=(40, 900), D=D, gamma=total, cap_slack=q_len, W=96, seed=4242 + D)
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    ws = wm.Workspace(cfg.batch * q_len, cfg.Hq, cfg.Hkv, cfg.D)
    wm.wmtp_ring_init_from_kv(dw.ring, dw.kv)
    orcs = [oracle_for(wl, b, with_ring=False) for b in range(cfg.batch)]
    i = 0
    for cyc, (d, with_full) in enumerate(cycles):
        # ---- extend: q_len tokens appended, then attended in one launch per variant
        sl = slice(i, i + q_len)
        km, vm, qm = (to_dev_bf16(_per_seq(a[sl])) for a in (wl.k_new, wl.v_new, wl.q))
        wm.wmtp_ring_append_many(dw.ring, km, vm)
        wm.wmtp_kv_append_many(dw.kv, km, vm, ws)
        out_w, out_f = torch.full_like(qm, float("nan")), torch.full_like(qm, float("nan"))
        lse_w = torch.full(qm.shape[:-1], float("nan"), dtype=torch.float32, device="cuda")
        lse_f = torch.full_like(lse_w, float("nan"))
        wm.wmtp_draft_extend_windowed(qm, dw.ring, out_w, ws, lse=lse_w)
        wm.wmtp_draft_extend_full(qm, dw.kv, out_f, ws, lse=lse_f)
        wm.wmtp_device_status(ws)
        for b in range(cfg.batch):
            for j in range(q_len):
                r = orcs[b].step(wl.q[i + j, b], wl.k_new[i + j, b], wl.v_new[i + j, b])
                compare(out_w[b, j], lse_w[b, j], *r["win"], what=f"cycle {cyc} extend windowed seq {b} token {j}")
                compare(out_f[b, j], lse_f[b, j], *r["full"], what=f"cycle {cyc} extend full seq {b} token {j}")
        i += q_len
        # ---- d decode steps on the same workspace
        sl = slice(i, i + d)
        q, kn, vn = dw.q[sl], dw.k_new[sl], dw.v_new[sl]
        ow, of = torch.full_like(q, float("nan")), torch.full_like(q, float("nan"))
        lw = torch.full(q.shape[:-1], float("nan"), dtype=torch.float32, device="cuda")
        lf = torch.full_like(lw, float("nan"))
        wm.wmtp_draft_loop_windowed(dw.ring, q, kn, vn, ow, ws, lse=lw)
        if with_full:
            wm.wmtp_draft_loop_full(dw.kv, q, kn, vn, of, ws, lse=lf)
        else:
            wm.wmtp_kv_append_many(dw.kv, to_dev_bf16(_per_seq(wl.k_new[sl])), to_dev_bf16(_per_seq(wl.v_new[sl])), ws)
        wm.wmtp_device_status(ws)
        for b in range(cfg.batch):
            for j in range(d):
                r = orcs[b].step(wl.q[i + j, b], wl.k_new[i + j, b], wl.v_new[i + j, b], full=with_full)
                compare(ow[j, b], lw[j, b], *r["win"], what=f"cycle {cyc} decode windowed seq {b} step {j}")
                if with_full:
                    compare(of[j, b], lf[j, b], *r["full"], what=f"cycle {cyc} decode full seq {b} step {j}")
        i += d
    assert all(int(dw.ring.len[b]) == orcs[b].S and int(dw.lens[b]) == orcs[b].S for b in range(cfg.batch))


def test_one_workspace_serves_two_batch_sizes_in_turn():
    """Two stores of different batch size share one workspace (sized for the larger); runs of odd and even length
    alternate, so a large launch meets per-segment words that only smaller launches have prepared since."""
    big = _cfg(name="big", batch=4, S0=0, S0_range=(30, 1200), D=128, gamma=8, W=64, seed=515)
    small = _cfg(name="small", batch=1, S0=700, D=128, gamma=8, W=64, seed=516)
    wls = {c.name: wi.make_workload(c) for c in (big, small)}
    dws = {n: DeviceWorkload(w) for n, w in wls.items()}
    ws = wm.Workspace(big.batch, big.Hq, big.Hkv, big.D)
    orcs = {n: [oracle_for(w, b, with_ring=False) for b in range(w.cfg.batch)] for n, w in wls.items()}
    done = {"big": 0, "small": 0}
    for dw in dws.values():
        wm.wmtp_ring_init_from_kv(dw.ring, dw.kv)
    for name, steps in (("big", 3), ("small", 3), ("big", 3), ("small", 1), ("big", 2), ("small", 2)):
        dw, wl, i = dws[name], wls[name], done[name]
        sl = slice(i, i + steps)
        q = dw.q[sl]
        ow = torch.full_like(q, float("nan"))
        lw = torch.full(q.shape[:-1], float("nan"), dtype=torch.float32, device="cuda")
        wm.wmtp_draft_loop_windowed(dw.ring, q, dw.k_new[sl], dw.v_new[sl], ow, ws, lse=lw)
        wm.wmtp_device_status(ws)
        for b in range(wl.cfg.batch):
            for j in range(steps):
                r = orcs[name][b].step(wl.q[i + j, b], wl.k_new[i + j, b], wl.v_new[i + j, b], full=False)
                compare(ow[j, b], lw[j, b], *r["win"], what=f"{name} step {i + j} seq {b}")
        done[name] += steps


# ------------------------------------------------------------------------------------------ snapshot / restore
@pytest.mark.parametrize("kv_dtype", ["bf16", "fp8"])
@pytest.mark.parametrize("where", ["device", "pinned host"])
def test_ring_snapshot_restores_a_ring_that_continues_bit_identically(kv_dtype, where):
    """Three draft steps, snapshot, two more steps; a second ring restored from the snapshot and given the same two steps
    ends with the same bits in every array and gave the same outputs; the blob's bytes beyond the state are untouched."""
    cfg = _cfg(S0=500, D=128, W=64, gamma=5, cap_slack=3, seed=4242, kv_dtype=kv_dtype,
               key_scale=(0.5, 2.0) if kv_dtype == "fp8" else None)
    wl = wi.make_workload(cfg)
    dw = DeviceWorkload(wl)
    wm.wmtp_ring_init_from_kv(dw.ring, dw.kv)
    need = wm.wmtp_ring_state_bytes(dw.ring)
    blob = torch.full((need + 512,), 0x5A, dtype=torch.uint8, device="cuda" if where == "device" else "cpu")
    if where != "device":
        blob = blob.pin_memory()
    q, kn, vn = dw.q, dw.k_new, dw.v_new
    outs = torch.full_like(q, float("nan"))
    wm.wmtp_draft_loop_windowed(dw.ring, q[:3], kn[:3], vn[:3], outs[:3], dw.ws)
    wm.wmtp_ring_export(dw.ring, blob)
    wm.wmtp_draft_loop_windowed(dw.ring, q[3:], kn[3:], vn[3:], outs[3:], dw.ws)
    torch.cuda.synchronize()
    assert (blob[need:] == 0x5A).all()
    twin = wm.Ring(cfg.batch, cfg.Hkv, cfg.D, cfg.n_sink, cfg.W, cap=cfg.W + cfg.cap_slack, k_scale=dw.k_scale, v_scale=dw.v_scale)
    twin.k.fill_(3); twin.v.fill_(3)                              # stale contents the import must replace
    wm.wmtp_ring_import(twin, blob)
    outs2 = torch.full_like(q[3:], float("nan"))
    wm.wmtp_draft_loop_windowed(twin, q[3:], kn[3:], vn[3:], outs2, dw.ws)
    wm.wmtp_device_status(dw.ws)
    dw.guard.check(cfg.name)
    assert torch.equal(bits_t(twin.k), bits_t(dw.ring.k)) and torch.equal(bits_t(twin.v), bits_t(dw.ring.v))
    assert torch.equal(twin.slot_pos, dw.ring.slot_pos) and torch.equal(twin.len, dw.ring.len)
    assert torch.equal(outs2.view(torch.int16), outs[3:].view(torch.int16))
    # and the continued ring is the oracle's ring
    orc = oracle_for(wl, 0)
    for i in range(cfg.gamma):
        r = orc.step(wl.q[i, 0], wl.k_new[i, 0], wl.v_new[i, 0], full=False)
        if i >= 3:
            compare(outs2[i - 3, 0], None, *r["win"], what=f"restored ring step {i}")
    check_ring_against_sim(twin, 0, orc.ring, "restored ring")


def bits_t(t):
    return t if t.dtype == torch.uint8 else t.view(torch.int16)


# ------------------------------------------------------------------------------------------ seeded random shapes
@pytest.mark.parametrize("idx", range(20))
def test_extend_random_shape(idx):
    """Draft-extend (windowed and full-context, multi-query kernel and per-query path alike) on seeded random shapes:
    group sizes that leave MMA columns empty, 1 to 9 sequences, 2 to 7 new tokens (one or two passes of four queries),
    both store types and layouts, CTA caps."""
    rs = np.random.RandomState(4100 + idx)
    Hkv = int(rs.choice([1, 2, 4]))
    G = int(rs.choice([1, 2, 3, 4, 7, 8]))
    q_len = int(rs.choice([2, 3, 4, 5, 7]))
    kv_dtype = str(rs.choice(["bf16", "fp8"]))
    cfg = wi.DraftConfig(
        name=f"extrand{idx}", batch=int(rs.choice([1, 1, 2, 3, 9])), S0=0, Hq=G * Hkv, Hkv=Hkv, D=int(rs.choice([128, 256])),
        W=int(rs.choice([16, 64, 200, 1024])), n_sink=int(rs.choice([0, 1, 4, 64])), gamma=q_len, seed=4200 + idx,
        S0_range=(1, int(rs.choice([200, 3000, 30000]))), paged=bool(rs.randint(2)), cap_slack=q_len - 1 + int(rs.choice([0, 3])),
        kv_dtype=kv_dtype, key_scale=(0.5, 2.0) if Hkv > 1 and rs.randint(2) else None)
    _extend_and_check(cfg, max_ctas=int(rs.choice([0, 0, 1, 5, 64])))
