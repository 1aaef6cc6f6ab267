"""The allocation-free windowed attention entry point.

Some users of this library cannot allocate device memory for a workspace: they run inside a runtime
that owns the allocator, or under a memory budget fixed at start-up. wmtp_draft_attn_windowed_noalloc
serves them from a fixed scratch array inside the library; it must give the same result as
wmtp_draft_attn_windowed, call after call, although the array is shared by every call and keeps the
previous call's contents -- whatever shape that call had. Checked against the workspace entry point
and against the CPU oracle.
Collected last on purpose (file name), so a stop-at-first-failure run has finished every other test.
"""
import pytest
import torch

import paper_2607_21535_b200 as wm
import wmtp_inputs as wi

from harness import DeviceWorkload, compare, oracle_for

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _defaults():
    wm.wmtp_set_max_ctas(0)
    wm.wmtp_set_work_stealing(True)
    yield
    wm.wmtp_set_max_ctas(0)


def _cfg(**kw):
    base = dict(name="noalloc", batch=2, S0=0, S0_range=(300, 3000), Hq=16, Hkv=2, D=256, W=512, n_sink=4, gamma=2,
                seed=2024)
    base.update(kw)
    return wi.DraftConfig(**base)


class _Case:
    """One store with its oracle; `step()` appends a token, runs the no-alloc call and checks it both ways."""

    def __init__(self, cfg, cap=None):
        self.cfg, self.wl = cfg, wi.make_workload(cfg)
        self.dw = DeviceWorkload(self.wl, cap=cap)
        wm.wmtp_ring_init_from_kv(self.dw.ring, self.dw.kv)
        self.orcs = [oracle_for(self.wl, b, cap=cap, with_ring=False) for b in range(cfg.batch)]
        self.i = 0

    def step(self, against_workspace=True):
        cfg, dw, i = self.cfg, self.dw, self.i
        shape = (cfg.batch, cfg.Hq, cfg.D)
        wm.wmtp_ring_append(dw.ring, dw.k_new[i], dw.v_new[i])
        got = torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        got_lse = torch.full(shape[:2], float("nan"), device="cuda")
        wm.wmtp_draft_attn_windowed_noalloc(dw.q[i], dw.ring, got, lse=got_lse)
        dw.guard.check(cfg.name)
        for b in range(cfg.batch):
            r = self.orcs[b].step(self.wl.q[i, b], self.wl.k_new[i, b], self.wl.v_new[i, b], full=False)
            compare(got[b], got_lse[b], *r["win"], what=f"{cfg.name} call {i} seq {b} vs oracle")
        if against_workspace:
            ref = torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda")
            ref_lse = torch.full(shape[:2], float("nan"), device="cuda")
            wm.wmtp_draft_attn_windowed(dw.q[i], dw.ring, ref, dw.ws, lse=ref_lse)
            wm.wmtp_device_status(dw.ws)
            d = (got.float() - ref.float()).abs()
            assert d.max().item() <= 2e-2 and d.mean().item() <= 2e-3          # the tolerance of the parity tests
            assert (got_lse - ref_lse).abs().max().item() <= 1e-3
            # same kernels on the same bits: equal up to the order in which split-KV partials are summed
            assert d.max().item() <= 4e-3
        self.i += 1


@pytest.mark.parametrize("D", [256, 128])
def test_noalloc_matches_workspace_entry_point_and_oracle_twice_in_a_row(D):
    case = _Case(_cfg(D=D))
    for _ in range(2):                                           # two calls in a row, ring advanced in between
        case.step()


def test_noalloc_at_the_limit_of_its_scratch():
    """batch * Hkv = 32 (the most the built-in scratch accepts) with 8 query heads per KV head and head_dim 256:
    ragged lengths, one ring still filling (not yet wrapped), one sequence that holds a single token."""
    cfg = _cfg(name="noalloc_limit", batch=16, S0_range=(300, 2500), W=384, gamma=3, seed=7)
    case = _Case(cfg)
    # make the extremes certain whatever the seeded lengths are: sequence 0 empty before its first append,
    # sequence 1 shorter than sink + window
    case.dw.lens[0] = 0
    case.dw.lens[1] = 100
    wm.wmtp_ring_init_from_kv(case.dw.ring, case.dw.kv)
    case.orcs[0] = _truncated_oracle(case.wl, 0, 0)
    case.orcs[1] = _truncated_oracle(case.wl, 1, 100)
    for _ in range(cfg.gamma):
        case.step()


def _truncated_oracle(wl, b, S):
    from oracle import reference as R
    cfg = wl.cfg
    return R.DraftOracle(wl.K[b][:, :S], wl.V[b][:, :S], cfg.Hq, cfg.n_sink, cfg.W, cap=cfg.W + cfg.cap_slack,
                         reserve=4 * cfg.gamma + 4, with_ring=False, k_scale=wl.k_scale, v_scale=wl.v_scale)


def test_noalloc_fp8_ring_and_ring_with_slack():
    a = _Case(_cfg(name="noalloc_fp8", kv_dtype="fp8", D=128, seed=11))
    b = _Case(_cfg(name="noalloc_slack", batch=3, W=200, cap_slack=9, seed=12), cap=209)
    for _ in range(2):
        a.step()
        b.step()


def test_noalloc_calls_of_differing_shape_share_the_scratch():
    """A run of calls whose (batch * Hkv) goes up and down: the array keeps the previous call's words, a larger call
    must not trip over what a smaller or larger one left behind."""
    small = _Case(_cfg(name="noalloc_b1", batch=1, gamma=4, seed=21))
    wide = _Case(_cfg(name="noalloc_b8", batch=8, Hq=32, Hkv=4, D=128, W=256, S0_range=(20, 1500), gamma=4, seed=22))
    mid = _Case(_cfg(name="noalloc_b5", batch=5, gamma=4, seed=23))
    for case in (wide, small, small, small, wide, mid, wide, small, mid, mid, wide):
        if case is wide and case.i == 3:
            case.step(against_workspace=False)
        else:
            case.step()


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
