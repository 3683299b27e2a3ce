"""The bounded device-side waits: a wait that runs out ends its thread block in an orderly way, raises the
device flag that unigist_device_status reports, and leaves the GPU usable.  The wait that runs out belongs to a
self-check block of the library (a barrier nothing completes): nothing faults and nothing hangs."""
import pytest
import torch

import paper_2509_15763_b200 as ug
from paper_2509_15763_b200 import synth

from gpu_util import run_attention

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_once_and_the_device_stays_usable():
    ug.unigist_device_status()  # nothing pending
    before = ug.unigist_launch_count()
    ug.unigist_selftest_wait_timeout()
    assert ug.unigist_launch_count() == before + 1
    with pytest.raises(ug.UnigistError) as err:
        ug.unigist_device_status()  # synchronises: the block has given up by now (about a second)
    assert err.value.code == 7  # UNIGIST_ERR_TIMEOUT
    assert "gave up" in ug.unigist_last_error_string()
    ug.unigist_device_status()  # the flag was cleared by the report
    # the context is intact: a forward + backward after it runs and is checked by its own status call
    w = synth.Workload("after_timeout", 1, 512, 8, 128, 4, 2, 128, seed=77)
    out = run_attention(w, backward=True)
    assert torch.isfinite(out["o"].float()).all() and torch.isfinite(out["dq"].float()).all()
