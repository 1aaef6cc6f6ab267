"""The give-up path of the kernels' bounded waits, exercised without faulting or hanging anything.

A CTA of the attention kernel that has published its partial of a (sequence, KV head) segment polls a global word
until the segment's other contributors have published theirs, for a limited number of polls. With the limit set to
one poll (a process-wide test knob) a launch whose CTAs share segments cannot satisfy that wait: the CTA gives up,
flags WMTP_ERR_DEVICE_TIMEOUT in the workspace and still runs to the end of the kernel, so the call returns and the
context stays usable. Nothing here traps, faults or waits without a bound."""
import pytest
import torch

import paper_2607_21535_b200 as wm
import wmtp_inputs as wi

from harness import DeviceWorkload, compare, oracle_for

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _restore_knobs():
    yield
    wm.wmtp_set_wait_limit(0)
    wm.wmtp_set_max_ctas(0)
    wm.wmtp_set_work_stealing(True)


def test_expired_wait_is_reported_and_the_workspace_recovers():
    # three CTAs over two long segments: CTA 1 works in both, so every segment has two contributors that finish
    # milliseconds of streaming apart -- the first to finish cannot see the other's partial at its one poll
    cfg = wi.DraftConfig(name="timeout", batch=1, S0=300_000, Hq=16, Hkv=2, D=128, W=256, n_sink=4, gamma=1, seed=99)
    wl = wi.make_workload(cfg, poison_unused=False)
    dw = DeviceWorkload(wl)
    q = dw.q[0]
    out = torch.full_like(q, float("nan"))
    lse = torch.full(q.shape[:-1], float("nan"), dtype=torch.float32, device="cuda")
    wm.wmtp_set_work_stealing(False)
    wm.wmtp_set_max_ctas(3)
    wm.wmtp_set_wait_limit(1)
    wm.wmtp_draft_attn_full(q, dw.kv, out, dw.ws, lse=lse)           # returns: every thread reaches the end of the kernel
    with pytest.raises(wm.WmtpError) as ei:
        wm.wmtp_device_status(dw.ws)
    assert ei.value.status == 6, ei.value
    # the sticky word was cleared by the read; the header says the workspace must be initialised again
    wm.wmtp_set_wait_limit(0)
    wm.wmtp_workspace_init(dw.ws)
    orc = oracle_for(wl, 0, with_ring=False)
    ref = orc.attend_full(wl.q[0, 0])
    for _ in range(2):                                               # twice: the launch epoch and both word copies work again
        out.fill_(float("nan")); lse.fill_(float("nan"))
        wm.wmtp_draft_attn_full(q, dw.kv, out, dw.ws, lse=lse)
        wm.wmtp_device_status(dw.ws)
        compare(out[0], lse[0], *ref, what="after re-initialising the workspace")
    # and with all CTAs and work stealing, as the library runs by default
    wm.wmtp_set_max_ctas(0)
    wm.wmtp_set_work_stealing(True)
    wm.wmtp_draft_attn_full(q, dw.kv, out, dw.ws, lse=lse)
    wm.wmtp_device_status(dw.ws)
    compare(out[0], lse[0], *ref, what="default configuration after the timeout")
