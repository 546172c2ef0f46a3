"""Failure detection without a GPU fault: a device-side wait that nothing satisfies runs out, the kernel returns
an error status that the host reads, and the context stays usable."""
import time

import numpy as np
import pytest
import torch

from paper_2510_08431_b200 import synth
from tests import gpu_util as U

pytestmark = pytest.mark.gpu


def test_bounded_wait_expires_and_reports(oracle):
    assert torch.cuda.is_available()
    from paper_2510_08431_b200 import build
    build.build_library()
    import paper_2510_08431_b200 as aj
    # a normal call first (creates the status word), with a clean status
    w = synth.WORKLOADS["tiny"]
    x = synth.make_workload(w)
    g = U.to_gpu(x)
    U.run(aj, g, w.scale)
    t0 = time.time()
    assert aj.attn_jvp_selftest_bounded_wait(torch.cuda.current_stream().cuda_stream) == 0
    torch.cuda.synchronize()                    # returns: the wait is bounded
    dt = time.time() - t0
    assert 0.5 < dt < 30.0, dt
    assert aj.attn_jvp_device_status() == aj.attn_jvp.ERR_DEVICE_TIMEOUT
    assert aj.attn_jvp_device_status() == 0     # reading clears it
    # the device is still usable and results are still right
    o, to, lse = U.run(aj, g, w.scale)
    U.check_all(oracle, aj, x, w.B, w.H, w.Lq, w.Lk, w.D, w.scale, np.arange(w.B * w.H * w.Lq), o, to, lse)
