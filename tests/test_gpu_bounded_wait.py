"""The error path that every device-side wait of the library shares: a wait on a barrier that nothing signals gives up
after its poll limit, the status word says ESC_DEV_TIMEOUT, and the context stays usable (no trap, no fault)."""
import time

import numpy as np
import pytest

from paper_2503_06671_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu


def test_bounded_wait_runs_out_and_the_library_carries_on(oracle):
    import torch

    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    import paper_2503_06671_b200 as pkg

    B, C, C_a, H, W, K = 1, 32, 16, 40, 72, 13
    ws = pkg.new_workspace(B, C_a, H, W, K)
    assert pkg.esc_convattn_device_status(ws) == 0
    t0 = time.time()
    pkg.esc_convattn_selftest_bounded_wait(ws)
    assert pkg.esc_convattn_device_status(ws) == 8            # synchronises: the wait has given up by then
    assert time.time() - t0 < 30.0
    assert "0x5e1f0000" in pkg.esc_last_error().lower()        # where it gave up
    assert pkg.esc_convattn_device_status(ws) == 0            # reported once, then cleared
    # the same workspace and context still work
    d = synth.make_inputs(B, C, C_a, H, W, K, synth.BF16, seed=4, channel_means=True)
    x = util.to_device(d["x"], synth.BF16, synth.NHWC)
    wl, wd, bd = util.weights_to_device(d, synth.BF16)
    out = torch.empty_like(x)
    pkg.esc_convattn_forward_ex(x, C_a, K, wl, wd, bd, out, util.layout_code(synth.NHWC), ws)
    torch.cuda.synchronize()
    assert pkg.esc_convattn_device_status(ws) == 0
    ref, mag = oracle.forward(d["x"], C_a, d["w_large"], d["w_dyn"], d["b_dyn"], want_mag=True)
    got = util.to_host_nchw(out, synth.NHWC)
    util.check_attention(got[:, :C_a], ref[:, :C_a], mag, synth.BF16, what="after the timed-out wait")
    assert np.array_equal(got[:, C_a:], ref[:, C_a:])
