"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle's own code.

Each test is chosen so that a plausible mistake in the oracle (a dropped scale, a wrong
sign, a transposed operand, an off-by-one in the window, a wrong GQA map) fails it.
"""
import math
import os

import numpy as np
import pytest

import wmtp_inputs as wi
from oracle import reference as R
from oracle import twin

BF = wi.f32_to_bf16_bits
F64 = wi.bf16_bits_to_f64


def _rand(seed, tid, shape, scale=1.0):
    return wi.normal_bf16(seed, tid, shape, scale=scale, threads=1)


# ---------------------------------------------------------------- golden fixtures (hand-worked)
def _read_golden(path):
    rows = []
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        rows.append(line)
    return rows


def test_keep_set_matches_hand_worked_examples(golden_dir):
    for line in _read_golden(os.path.join(golden_dir, "keep_sets.txt")):
        lhs, rhs = line.split(":")
        S, n_sink, W = (int(t) for t in lhs.split())
        want = [int(t) for t in rhs.split()]
        assert R.keep_set(S, n_sink, W) == want, line
        st = R.WindowStore(n_sink, W)
        for p in range(S):
            st.append(p, p)
        assert st.positions() == want, line


def test_kv_bytes_per_token_match_paper(golden_dir):
    for line in _read_golden(os.path.join(golden_dir, "kv_bytes.txt")):
        Hkv, D, nbytes = (int(t) for t in line.split())
        cfg = wi.scaled(wi.CONFIGS[2], Hkv=Hkv, D=D)
        assert cfg.kv_bytes_per_token == nbytes
    # the million-token configuration reads ~2 GB per full-context step, ~8 MB windowed
    c3 = wi.CONFIGS[2]
    assert c3.S0 * c3.kv_bytes_per_token == 2 << 30
    assert (c3.W + c3.n_sink) * c3.kv_bytes_per_token == 4100 * 2048


# ---------------------------------------------------------------- key set / stores, brute force
@pytest.mark.parametrize("n_sink,W", [(0, 1), (1, 1), (2, 3), (4, 8), (0, 5), (3, 1)])
def test_window_store_brute_force(n_sink, W):
    st = R.WindowStore(n_sink, W)
    for S in range(1, n_sink + W + 71):
        st.append(("k", S - 1), ("v", S - 1))
        brute = [p for p in range(S) if p < n_sink or p >= S - W]          # written independently
        assert st.positions() == brute
        assert R.keep_set(S, n_sink, W) == brute
        assert twin.window_positions(S, n_sink, W) == brute
        assert len(brute) == min(S, n_sink + W)                            # reads min(seq, W + n_sink) tokens
        assert all(e[1] == ("k", e[0]) and e[2] == ("v", e[0]) for e in st.entries())


@pytest.mark.parametrize("n_sink,W,slack", [(0, 1, 0), (1, 1, 0), (2, 3, 0), (4, 8, 0), (4, 8, 3), (2, 5, 7)])
def test_ring_sim_holds_sink_and_last_W(n_sink, W, slack):
    cap = W + slack
    Hkv, D = 2, 4
    ring = R.RingSim(n_sink, cap, Hkv, D)
    rows = {}
    for p in range(3 * (n_sink + cap) + 6):
        k = np.full((Hkv, D), p * 2 + 1, dtype=np.uint16)
        v = np.full((Hkv, D), p * 2 + 2, dtype=np.uint16)
        rows[p] = (k, v)
        slot = ring.append(k, v)
        S = p + 1
        # footprint independent of S; closed-form slot (sink fixed, window region circular)
        assert slot == (p if p < n_sink else n_sink + (p - n_sink) % cap)
        assert ring.length == S
        held = {int(x) for x in ring.slot_pos if x >= 0}
        want = {q for q in range(S) if q < n_sink or q >= S - cap}
        assert held == want                                   # ring = sink U last `cap` tokens
        assert set(R.keep_set(S, n_sink, W)) <= held          # everything the draft reads is present
        for s, q in enumerate(ring.slot_pos):
            if q >= 0:
                assert (ring.K[:, s] == rows[int(q)][0]).all() and (ring.V[:, s] == rows[int(q)][1]).all()
            else:
                assert not ring.written[s]


@pytest.mark.parametrize("n_sink,W,d", [(4, 8, 3), (0, 5, 7), (2, 3, 1), (3, 6, 6)])
def test_ring_sim_rollback_within_slack_keeps_the_window(n_sink, W, d):
    """With d slack slots (Section 4 "Memory", Section 6 tree speculation: n_sink + W + d) up to d speculative tokens
    can be written and discarded: afterwards the ring still holds every position of sink + last W, with the rows the
    positions were first given, and appending again behaves as if the discarded tokens had never been written."""
    cap, Hkv, D = W + d, 1, 2
    rng = np.random.RandomState(n_sink * 100 + W)
    ring, clean = R.RingSim(n_sink, cap, Hkv, D), R.RingSim(n_sink, cap, Hkv, D)
    row = lambda p, gen: np.full((Hkv, D), (p * 7 + gen * 3 + 1) % 65521, dtype=np.uint16)
    S = 0
    for it in range(60):
        n_acc, n_rej = int(rng.randint(0, 4)), int(rng.randint(0, d + 1))
        for _ in range(n_acc):                                 # tokens that stay: both rings get them
            ring.append(row(S, 0), row(S, 0)); clean.append(row(S, 0), row(S, 0)); S += 1
        for j in range(n_rej):                                 # speculative tokens: only the ring with rollback sees them
            ring.append(row(S + j, it + 1), row(S + j, it + 1))
        ring.rewind(n_rej)
        assert ring.length == clean.length == S
        held = {int(p): s for s, p in enumerate(ring.slot_pos) if p >= 0}
        assert all(p < S for p in held)                        # no slot claims a discarded position
        for p in R.keep_set(S, n_sink, W):                     # brute force over what the draft reads
            s = held[p]
            assert s == (p if p < n_sink else n_sink + (p - n_sink) % cap)
            assert ring.written[s] and (ring.K[:, s] == row(p, 0)).all() and (ring.V[:, s] == row(p, 0)).all()
        # the next append lands where it would have without the speculation
        assert ring.append(row(S, 0), row(S, 0)) == clean.append(row(S, 0), row(S, 0)); S += 1


# ---------------------------------------------------------------- softmax attention, closed forms
def test_uniform_keys_give_mean_of_values():
    Hq, Hkv, D, n = 8, 2, 16, 37
    q = _rand(1, 1, (Hq, D))
    krow = _rand(1, 2, (Hkv, 1, D))
    K = np.repeat(krow, n, axis=1)
    V = _rand(1, 3, (Hkv, n, D))
    out, lse = R.attention(q, K, V)
    G = Hq // Hkv
    for h in range(Hq):
        g = h // G
        np.testing.assert_allclose(out[h], F64(V[g]).mean(axis=0), rtol=0, atol=1e-13)
        z = (F64(q[h]) * F64(krow[g, 0])).sum() / math.sqrt(D)
        assert abs(lse[h] - (z + math.log(n))) < 1e-12


def test_zero_query_gives_mean_and_log_count():
    Hq, Hkv, D, n = 4, 4, 8, 11
    q = np.zeros((Hq, D), dtype=np.uint16)
    K, V = _rand(2, 2, (Hkv, n, D)), _rand(2, 3, (Hkv, n, D))
    out, lse = R.attention(q, K, V)
    for h in range(Hq):
        np.testing.assert_allclose(out[h], F64(V[h]).mean(axis=0), atol=1e-14)
        assert abs(lse[h] - math.log(n)) < 1e-14


def test_single_key_returns_its_value_exactly():
    Hq, Hkv, D = 6, 3, 8
    q, K, V = _rand(3, 1, (Hq, D)), _rand(3, 2, (Hkv, 1, D)), _rand(3, 3, (Hkv, 1, D))
    out, lse = R.attention(q, K, V)
    for h in range(Hq):
        g = h // 2
        assert (out[h] == F64(V[g, 0])).all()
        assert abs(lse[h] - (F64(q[h]) * F64(K[g, 0])).sum() / math.sqrt(D)) < 1e-14


def test_two_keys_logistic_closed_form_and_scale():
    # q = 4*e_0 ; k_a = 3*e_0, k_b = -1*e_0 ; logits = scale*12, scale*(-4).
    D = 4
    q = BF(np.array([[4, 0, 0, 0]], dtype=np.float32))
    K = BF(np.array([[[3, 9, 9, 9], [-1, 5, 5, 5]]], dtype=np.float32))
    V = BF(np.array([[[1, 0, 2, 8], [0, 1, -2, 4]]], dtype=np.float32))
    for scale in (None, 0.125, 1.0):
        s = 1 / math.sqrt(D) if scale is None else scale
        out, lse = R.attention(q, K, V, sm_scale=scale)
        wa = 1.0 / (1.0 + math.exp(-(12 * s - (-4 * s))))       # logistic of the logit gap
        want = wa * np.array([1, 0, 2, 8.0]) + (1 - wa) * np.array([0, 1, -2, 4.0])
        np.testing.assert_allclose(out[0], want, rtol=1e-14, atol=1e-15)
        assert abs(lse[0] - (12 * s + math.log1p(math.exp(-16 * s)))) < 1e-13


def test_dominant_key_wins():
    Hq, Hkv, D, n = 4, 1, 16, 50
    q = BF(np.ones((Hq, D), dtype=np.float32) * 2)
    Kf = np.zeros((Hkv, n, D), dtype=np.float32)
    Kf[0, 17] = 8.0                                   # logit 2*8*16/4 = 64 above the rest (0)
    K, V = BF(Kf), _rand(4, 3, (Hkv, n, D))
    out, lse = R.attention(q, K, V)
    np.testing.assert_allclose(out, np.broadcast_to(F64(V[0, 17]), (Hq, D)), atol=1e-20 + 50 * math.exp(-64) * 5)
    np.testing.assert_allclose(lse, 64.0, atol=1e-12)


def test_gqa_head_map_is_consecutive_groups():
    Hq, Hkv, D, n = 8, 4, 4, 5
    q = _rand(5, 1, (Hq, D))
    K = _rand(5, 2, (Hkv, n, D))
    Vf = np.zeros((Hkv, n, D), dtype=np.float32)
    for g in range(Hkv):
        Vf[g] = g + 1
    out, _ = R.attention(q, K, BF(Vf))
    np.testing.assert_allclose(out[:, 0], [1, 1, 2, 2, 3, 3, 4, 4], atol=1e-14)


def test_shift_and_permutation_invariance():
    Hq, Hkv, D, n = 4, 2, 8, 23
    rs = np.random.RandomState(0)
    q = BF(rs.randint(-3, 4, (Hq, D)).astype(np.float32))
    Kf = rs.randint(-4, 5, (Hkv, n, D)).astype(np.float32)
    c = rs.randint(-2, 3, (Hkv, 1, D)).astype(np.float32)
    V = _rand(6, 3, (Hkv, n, D))
    o0, l0 = R.attention(q, BF(Kf), V)
    o1, l1 = R.attention(q, BF(Kf + c), V)                       # K + c exact in bf16 (small integers)
    np.testing.assert_allclose(o1, o0, atol=1e-13)
    for h in range(Hq):
        shift = (F64(q[h]) * c[h // 2, 0]).sum() / math.sqrt(D)
        assert abs((l1[h] - l0[h]) - shift) < 1e-12
    perm = rs.permutation(n)
    o2, l2 = R.attention(q, BF(Kf), V, keys=perm)
    np.testing.assert_allclose(o2, o0, atol=1e-14)
    np.testing.assert_allclose(l2, l0, atol=1e-14)
    # a strict subset lowers lse and equals attention over the gathered rows
    sub = np.sort(perm[: n // 2])
    o3, l3 = R.attention(q, BF(Kf), V, keys=sub)
    o4, l4 = R.attention(q, np.ascontiguousarray(BF(Kf)[:, sub]), np.ascontiguousarray(V[:, sub]))
    assert (o3 == o4).all() and (l3 == l4).all() and (l3 < l0).all()


def test_empty_key_set():
    q = _rand(7, 1, (2, 4))
    K = np.zeros((1, 0, 4), dtype=np.uint16)
    out, lse = R.attention(q, K, K)
    assert (out == 0).all() and np.isneginf(lse).all()


# ---------------------------------------------------------------- brute force and library cross-check
@pytest.mark.parametrize("n", [1, 2, 7, 33, 64])
def test_against_pure_python_twin(n):
    Hq, Hkv, D = 4, 2, 8
    q, K, V = _rand(8, (1, n), (Hq, D)), _rand(8, (2, n), (Hkv, n, D), scale=2.0), _rand(8, (3, n), (Hkv, n, D))
    out, lse = R.attention(q, K, V, sm_scale=0.3)
    o_py, l_py = twin.attention_py(q.tolist(), K.tolist(), V.tolist(), Hq // Hkv, 0.3)
    np.testing.assert_allclose(out, np.array(o_py), rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(lse, np.array(l_py), rtol=1e-13, atol=1e-13)


def test_against_torch_sdpa_fp64():
    import torch
    Hq, Hkv, D, n = 16, 2, 128, 777
    q, K, V = _rand(9, 1, (Hq, D)), _rand(9, 2, (Hkv, n, D)), _rand(9, 3, (Hkv, n, D))
    out, lse = R.attention(q, K, V)
    tq = torch.from_numpy(F64(q)).view(1, Hq, 1, D)
    tk = torch.from_numpy(F64(K)).repeat_interleave(Hq // Hkv, dim=0).unsqueeze(0)
    tv = torch.from_numpy(F64(V)).repeat_interleave(Hq // Hkv, dim=0).unsqueeze(0)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv)[0, :, 0, :].numpy()
    np.testing.assert_allclose(out, ref, rtol=1e-11, atol=1e-13)
    z = (tq @ tk.transpose(-1, -2))[0, :, 0, :] / math.sqrt(D)
    np.testing.assert_allclose(lse, torch.logsumexp(z, dim=-1).numpy(), rtol=1e-13)


# ---------------------------------------------------------------- windowed vs full relations
def _small_cfg(**kw):
    base = dict(name="t", batch=1, S0=40, Hq=4, Hkv=2, D=16, W=8, n_sink=2, gamma=3, seed=77)
    base.update(kw)
    return wi.DraftConfig(**base)


@pytest.mark.parametrize("S0", [0, 1, 2, 5, 7])
def test_windowed_equals_full_when_window_covers_context(S0):
    cfg = _small_cfg(S0=S0)          # S0 + gamma <= n_sink + W = 10
    wl = wi.make_workload(cfg, threads=1)
    o = R.DraftOracle(wl.K[0], wl.V[0], cfg.Hq, cfg.n_sink, cfg.W)
    for i in range(cfg.gamma):
        r = o.step(wl.q[i, 0], wl.k_new[i, 0], wl.v_new[i, 0])
        assert (r["win"][0] == r["full"][0]).all() and (r["win"][1] == r["full"][1]).all()


def test_windowed_store_equals_keep_set_applied_to_full_kv():
    cfg = _small_cfg(S0=61)
    wl = wi.make_workload(cfg, threads=1)
    o = R.DraftOracle(wl.K[0], wl.V[0], cfg.Hq, cfg.n_sink, cfg.W)
    for i in range(cfg.gamma):
        r = o.step(wl.q[i, 0], wl.k_new[i, 0], wl.v_new[i, 0])
        keep = R.keep_set(o.S, cfg.n_sink, cfg.W)
        ow, lw = R.attention(wl.q[i, 0], o.Kfull[:, : o.S], o.Vfull[:, : o.S], keys=keep)
        np.testing.assert_allclose(r["win"][0], ow, atol=1e-15)
        np.testing.assert_allclose(r["win"][1], lw, atol=1e-15)
        # the ring simulation holds exactly the rows the store holds
        held = {int(p): s for s, p in enumerate(o.ring.slot_pos) if p >= 0}
        assert sorted(held) == keep
        for p in keep:
            assert (o.ring.K[:, held[p]] == o.Kfull[:, p]).all() and (o.ring.V[:, held[p]] == o.Vfull[:, p]).all()


def test_mass_identity_and_needle():
    cfg = _small_cfg(S0=300, W=32, n_sink=4, D=32)
    wl = wi.make_workload(cfg, threads=1)
    K0, V0 = wl.K[0].copy(), wl.V[0].copy()
    # plant a far key aligned with query head 0 of step 0 (outside sink and window)
    qf = wi.bf16_bits_to_f32(wl.q[0, 0, 0])
    K0[0, 100] = BF(qf * 3.0)
    o = R.DraftOracle(K0, V0, cfg.Hq, cfg.n_sink, cfg.W)
    r = o.step(wl.q[0, 0], wl.k_new[0, 0], wl.v_new[0, 0])
    (ow, lw), (of, lf) = r["win"], r["full"]
    S = o.S
    keep = set(R.keep_set(S, cfg.n_sink, cfg.W))
    far = [p for p in range(S) if p not in keep]
    ofar, lfar = R.attention(wl.q[0, 0], o.Kfull[:, :S], o.Vfull[:, :S], keys=far)
    mu = R.in_window_mass(lw, lf)
    assert ((mu > 0) & (mu <= 1)).all() and (lw <= lf).all()
    np.testing.assert_allclose(mu + np.exp(lfar - lf), 1.0, atol=1e-13)            # Z_win/Z + Z_far/Z = 1
    np.testing.assert_allclose(of, mu[:, None] * ow + (1 - mu)[:, None] * ofar, atol=1e-13)
    # head 0 of the full read-out is pulled to the needle's value row; the windowed one is not
    needle_v = F64(V0[0, 100])
    assert mu[0] < 1e-3
    assert np.abs(of[0] - needle_v).max() < 1e-2
    assert np.abs(ow[0] - needle_v).max() > 0.5
    assert R.win_perturb(of, ow)[0] > 0.5


def test_tail_out_frac_matches_far_key_contribution():
    cfg = _small_cfg(S0=200, W=24, n_sink=3, D=16)
    wl = wi.make_workload(cfg, threads=1)
    o = R.DraftOracle(wl.K[0], wl.V[0], cfg.Hq, cfg.n_sink, cfg.W)
    r = o.step(wl.q[0, 0], wl.k_new[0, 0], wl.v_new[0, 0])
    (ow, lw), (of, lf) = r["win"], r["full"]
    keep = set(R.keep_set(o.S, cfg.n_sink, cfg.W))
    far = [p for p in range(o.S) if p not in keep]
    ofar, lfar = R.attention(wl.q[0, 0], o.Kfull[:, :o.S], o.Vfull[:, :o.S], keys=far)
    far_share = np.exp(lfar - lf)[:, None] * ofar                 # the far keys' part of the full read-out, computed directly
    want = np.linalg.norm(far_share, axis=-1) / np.linalg.norm(of, axis=-1)
    np.testing.assert_allclose(R.tail_out_frac(of, ow, lw, lf), want, rtol=1e-10)
    # dropping nothing changes nothing
    np.testing.assert_allclose(R.tail_out_frac(of, of, lf, lf), 0.0, atol=1e-15)
    np.testing.assert_allclose(R.win_perturb(of, of), 0.0, atol=1e-15)


def test_win_perturb_is_the_difference_norm_over_the_full_norm():
    """Appendix D, caption of the attention-mass table: win_perturb = ||o_full - o_win|| / ||o_full||.
    Hand vectors fix numerator and denominator separately: a 3-4-5 triangle whose windowed read-out has
    another norm than the full one, so dividing by ||o_win|| (4/3) or by nothing (4) cannot pass."""
    assert R.win_perturb([3.0, 4.0], [3.0, 0.0]) == pytest.approx(4.0 / 5.0, abs=1e-15)
    assert R.win_perturb([3.0, 0.0], [3.0, 4.0]) == pytest.approx(4.0 / 3.0, abs=1e-15)     # not symmetric in its arguments
    assert R.win_perturb([0.0, 5.0], [0.0, -5.0]) == pytest.approx(2.0, abs=1e-15)          # a sign flip doubles, not cancels
    # rows are treated one by one (the last axis is the head dimension)
    got = R.win_perturb([[3.0, 4.0], [6.0, 8.0]], [[3.0, 0.0], [0.0, 8.0]])
    np.testing.assert_allclose(got, [0.8, 0.6], atol=1e-15)
    # on real oracle read-outs with ||o_win|| != ||o_full||: the norms written out as plain sums
    cfg = _small_cfg(S0=240, W=16, n_sink=2, D=16)
    wl = wi.make_workload(cfg, threads=1)
    o = R.DraftOracle(wl.K[0], wl.V[0], cfg.Hq, cfg.n_sink, cfg.W)
    r = o.step(wl.q[0, 0], wl.k_new[0, 0], wl.v_new[0, 0])
    (ow, _), (of, _) = r["win"], r["full"]
    got = R.win_perturb(of, ow)
    for h in range(cfg.Hq):
        num = math.sqrt(sum((float(of[h, d]) - float(ow[h, d])) ** 2 for d in range(cfg.D)))
        den_full = math.sqrt(sum(float(of[h, d]) ** 2 for d in range(cfg.D)))
        den_win = math.sqrt(sum(float(ow[h, d]) ** 2 for d in range(cfg.D)))
        assert abs(den_full - den_win) > 0.05 * den_full          # the case separates the two denominators
        assert got[h] == pytest.approx(num / den_full, rel=1e-12)
        assert abs(got[h] - num / den_win) > 1e-3


# ---------------------------------------------------------------- fp8 (e4m3) KV entries
def test_e4m3_decode_matches_hand_worked_codes(golden_dir):
    n = 0
    for line in _read_golden(os.path.join(golden_dir, "e4m3_codes.txt")):
        code, rest = line.split(None, 1)
        got = float(R.e4m3_decode(np.array([int(code, 16)], dtype=np.uint8))[0])
        if rest.strip() == "nan":
            assert math.isnan(got), line
        else:
            num, shift = rest.split("/")
            want = float(num) / 2.0 ** int(shift.strip()[2:])
            assert got == want and math.copysign(1.0, got) == math.copysign(1.0, float(num)), line
            assert int(code, 16) == int(R.e4m3_encode(np.float32([want]))[0]), line          # and back
        n += 1
    assert n >= 25


def test_e4m3_decode_matches_the_format_definition_and_torch():
    import torch
    codes = np.arange(256, dtype=np.uint8)
    val = R.e4m3_decode(codes)
    # hand-worked codes: zero, smallest subnormal, largest subnormal, smallest normal, one, 1.5, largest finite, NaN
    hand = {0x00: 0.0, 0x01: 2.0 ** -9, 0x07: 7 * 2.0 ** -9, 0x08: 2.0 ** -6, 0x38: 1.0, 0x3C: 1.5, 0x40: 2.0,
            0x7E: 448.0, 0x77: 240.0, 0xB8: -1.0, 0xFE: -448.0, 0x81: -(2.0 ** -9)}
    for c, v in hand.items():
        assert val[c] == v, hex(c)
    assert np.isnan(val[0x7F]) and np.isnan(val[0xFF]) and np.isfinite(np.delete(val, [0x7F, 0xFF])).all()
    assert np.signbit(val[0x80]) and val[0x80] == 0.0
    pos = val[:0x7F]
    assert (np.diff(pos) > 0).all()                                        # codes are ordered like their values
    assert (np.diff(pos)[:8] == 2.0 ** -9).all()                           # subnormal spacing continues into the first binade
    assert (val[0x80:0xFF] == -pos).all()
    lib_val = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.array_equal(np.isnan(val), np.isnan(lib_val)) and (val[~np.isnan(val)] == lib_val[~np.isnan(val)]).all()


def test_e4m3_encode_is_nearest_ties_to_even_and_saturates():
    import torch
    table = R.e4m3_decode(np.arange(0x7F, dtype=np.uint8))                 # the 127 non-negative finite values, ascending
    rs = np.random.RandomState(11)
    x = (rs.standard_normal(60000) * np.exp(rs.uniform(-14, 7, 60000))).astype(np.float32)
    mid = ((table[:-1] + table[1:]) / 2).astype(np.float32)                # exact ties (representable in fp32)
    x = np.concatenate([x, mid, -mid, table.astype(np.float32), np.float32([0.0, -0.0, 448, 449, 463.9, 464, 480, 1e9, -1e9,
                                                                              2.0 ** -10, 3 * 2.0 ** -10, 2.0 ** -11])])
    got = R.e4m3_encode(x)
    # brute force: nearest table entry, ties to the even code, beyond the table the last entry
    a = np.abs(x.astype(np.float64))
    dist = np.abs(a[:, None] - table[None, :])
    best = dist.min(axis=1)
    cand = dist == best[:, None]
    first = cand.argmax(axis=1)
    last = cand.shape[1] - 1 - cand[:, ::-1].argmax(axis=1)
    want = np.where(first == last, first, np.where(first % 2 == 0, first, last))
    want = want | (np.signbit(x).astype(np.int64) << 7)
    assert (got == want).all()
    assert (got[np.abs(x) >= 448] & 0x7F == 0x7E).all()                    # saturation, never NaN
    assert R.e4m3_encode(np.float32([np.nan]))[0] & 0x7F == 0x7F
    fin = np.array([c for c in range(256) if c & 0x7F != 0x7F], dtype=np.uint8)
    assert (R.e4m3_encode(R.e4m3_decode(fin).astype(np.float32)) == fin).all()      # every code is a fixed point
    m = np.abs(x) <= 448
    lib_codes = torch.from_numpy(x[m]).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert (got[m] == lib_codes).all()


def test_quantize_rows_divides_in_fp32():
    rs = np.random.RandomState(3)
    rows = wi.normal_bf16(9, 1, (3, 64))
    scale = np.float32([0.013, 0.7, 3.1])
    got = R.quantize_rows(rows, scale)
    x = (rows.astype(np.uint32) << 16).view(np.float32)
    for g in range(3):
        for d in range(64):
            t = np.float32(x[g, d]) / np.float32(scale[g])
            assert got[g, d] == R.e4m3_encode(np.float32([t]))[0]
    # dequantised value within half a code spacing (relative 2^-4) of the input, for inputs inside the range
    back = R.e4m3_decode(got) * scale[:, None].astype(np.float64)
    inside = np.abs(x) < 448 * scale[:, None]
    rel = np.abs(back - x)[inside] / np.maximum(np.abs(x[inside]), 2.0 ** -6 * np.repeat(scale, 64).reshape(3, 64)[inside])
    assert rel.max() <= 2.0 ** -4 + 1e-7


def test_fp8_attention_equals_bf16_attention_on_exactly_representable_values():
    """With power-of-two scales every dequantised entry is a bf16 value, so the fp8 read-out must equal the bf16
    read-out of those values; a single key returns code value * v_scale exactly for any scale."""
    rs = np.random.RandomState(5)
    Hq, Hkv, D, n = 8, 2, 32, 50
    q = wi.normal_bf16(21, 1, (Hq, D))
    codes_k = rs.randint(0, 256, (Hkv, n, D)).astype(np.uint8)
    codes_v = rs.randint(0, 256, (Hkv, n, D)).astype(np.uint8)
    codes_k[(codes_k & 0x7F) == 0x7F] = 0x30
    codes_v[(codes_v & 0x7F) == 0x7F] = 0x30
    codes_k = (codes_k & 0x80) | np.minimum(codes_k & 0x7F, 0x47)             # keep the logits moderate
    ks, vs = np.float32([2.0 ** -5, 2.0 ** -3]), np.float32([2.0 ** -7, 2.0 ** 1])
    Kf = (R.e4m3_decode(codes_k) * ks[:, None, None]).astype(np.float32)
    Vf = (R.e4m3_decode(codes_v) * vs[:, None, None]).astype(np.float32)
    Kb, Vb = (Kf.view(np.uint32) >> 16).astype(np.uint16), (Vf.view(np.uint32) >> 16).astype(np.uint16)
    assert ((Kb.astype(np.uint32) << 16).view(np.float32) == Kf).all()        # exactly representable
    keys = np.array([3, 17, 4, 44, 45, 9])
    o8, l8 = R.attention(q, codes_k, codes_v, keys=keys, k_scale=ks, v_scale=vs)
    ob, lb = R.attention(q, Kb, Vb, keys=keys)
    assert np.abs(o8 - ob).max() < 1e-12 and np.abs(l8 - lb).max() < 1e-12
    vs2 = np.float32([0.0371, 1.9])
    o1, _ = R.attention(q, codes_k, codes_v, keys=np.array([7]), k_scale=ks, v_scale=vs2)
    for h in range(Hq):
        assert (o1[h] == R.e4m3_decode(codes_v[h // 4, 7]) * np.float64(vs2[h // 4])).all()


def test_fp8_draft_oracle_quantises_on_append():
    cfg = wi.DraftConfig("f8pin", 1, 20, 8, 2, 32, 16, 4, 3, seed=77, kv_dtype="fp8", key_scale=(0.5, 2.0))
    wl = wi.make_workload(cfg)
    assert wl.K[0].dtype == np.uint8 and not (wl.K[0] & 0x7F == 0x7F).any()
    orc = R.DraftOracle(wl.K[0], wl.V[0], cfg.Hq, cfg.n_sink, cfg.W, k_scale=wl.k_scale, v_scale=wl.v_scale)
    r = orc.step(wl.q[0, 0], wl.k_new[0, 0], wl.v_new[0, 0])
    assert (orc.Kfull[:, 20] == R.quantize_rows(wl.k_new[0, 0], wl.k_scale)).all()
    assert (orc.ring.K[:, orc.ring.slot_pos.tolist().index(20)] == orc.Kfull[:, 20]).all()
    # S = 21 > n_sink + W = 20: windowed drops exactly position 4
    keep = R.keep_set(21, 4, 16)
    assert keep == [0, 1, 2, 3] + list(range(5, 21))
    ow, lw = R.attention(wl.q[0, 0], orc.Kfull[:, :21], orc.Vfull[:, :21], keys=np.array(keep), k_scale=wl.k_scale, v_scale=wl.v_scale)
    assert np.abs(ow - r["win"][0]).max() < 1e-12 and np.abs(lw - r["win"][1]).max() < 1e-12
    assert (r["full"][1] > r["win"][1]).all()


# ---------------------------------------------------------------- reduced block table
@pytest.mark.parametrize("n_sink,W,ps", [(4, 64, 64), (0, 100, 64), (64, 4032 // 16, 64), (70, 130, 64), (3, 5, 4), (4, 8, 16)])
def test_reduced_block_table_expands_to_the_keep_set(n_sink, W, ps):
    """Walking the reduced table with its row bounds must visit exactly the rows of the kept positions, in order."""
    rs = np.random.RandomState(n_sink + W)
    for S in list(range(0, 3 * ps + 3)) + [n_sink + W, n_sink + W + 1, 10 * ps - 1, 10 * ps, 10 * ps + 1, 977]:
        n_pages = (S + ps - 1) // ps + 2
        page_row = rs.permutation(n_pages + 50)[:n_pages]
        pages, meta = R.reduced_block_table(S, n_sink, W, page_row, ps)
        n_s, n_w, sink_last, win_first, win_last = meta
        assert len(pages) == n_s + n_w and n_s <= (n_sink + ps - 1) // ps and n_w <= (W + ps - 1) // ps + 1
        rows = []                                              # (page, row) pairs a reader would touch
        for i in range(n_s):
            hi = sink_last if i == n_s - 1 else ps
            rows += [(pages[i], r) for r in range(hi)]
        for i in range(n_w):
            lo = win_first if i == 0 else 0
            hi = win_last if i == n_w - 1 else ps
            rows += [(pages[n_s + i], r) for r in range(lo, hi)]
        want = [(int(page_row[p // ps]), p % ps) for p in R.keep_set(S, n_sink, W)]        # brute force, token by token
        assert rows == want, (S, meta)


@pytest.mark.parametrize("ps", [64, 16])
def test_full_token_index_gathers_the_logical_sequence_from_the_pool(ps):
    """The index is right when reading the pool through it gives back every sequence's keys in order: pool rows are
    filled from the logical K by the input generator's own scatter (page by page), the index must invert it."""
    cfg = wi.DraftConfig("idx", 3, 0, 4, 2, 128, 32, 2, 1, seed=5150 + ps, S0_range=(1, 5 * ps + 3), paged=True, page_size=ps)
    wl = wi.make_workload(cfg, poison_unused=False)
    pool = wl.K_dev                                              # [num_pages][Hkv][ps][D]
    rows = np.ascontiguousarray(np.swapaxes(pool, 0, 1)).reshape(cfg.Hkv, -1, cfg.D)     # per KV head: pool row -> key
    stride = int(wl.seq_lens.max()) + 5
    for b in range(cfg.batch):
        S = int(wl.seq_lens[b])
        idx = R.full_token_index(S, wl.page_table[b], ps, stride)
        assert len(idx) == stride and all(i == -1 for i in idx[S:]) and all(i >= 0 for i in idx[:S])
        assert len(set(idx[:S])) == S                            # no pool row twice
        for g in range(cfg.Hkv):
            assert (rows[g][idx[:S]] == wl.K[b][g][:S]).all()
    # a table shorter than the sequence keeps its first entries
    assert R.full_token_index(10, [7, 3], 4, 6) == [28, 29, 30, 31, 12, 13]
