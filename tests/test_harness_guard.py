"""The test harness's own guard bands: a write outside a guarded array must be noticed, writes inside must not."""
import pytest
import torch

from harness import GuardedAlloc


def test_guard_bands_notice_writes_before_and_after_an_array():
    for where in ("inside", "before", "after"):
        g = GuardedAlloc()
        t = g((3, 5), torch.int32, "cpu", "probe")
        t.fill_(7)                                            # every element of the array itself: allowed
        name, buf, off, nbytes = g.blocks[0]
        assert nbytes == 60 and (t == 7).all() and t.data_ptr() % 256 == 0
        if where == "before":
            buf[off - 1] = 0
        elif where == "after":
            buf[off + nbytes] = 0                             # the first byte past the array (inside its padding)
        if where == "inside":
            g.check("probe")
        else:
            with pytest.raises(AssertionError, match="outside probe"):
                g.check("probe")


def test_guarded_copy_keeps_contents_and_alignment():
    g = GuardedAlloc()
    src = torch.arange(1000, dtype=torch.int64)
    dst = g.like(src, "copy")
    assert torch.equal(src, dst) and dst.data_ptr() % 256 == 0
    g.check()
