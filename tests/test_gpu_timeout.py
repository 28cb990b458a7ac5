"""A bounded device-side wait that runs out: the kernel must return, report it, and leave the GPU usable.

Every spin-wait in the kernels gives up after a cycle limit; the thread that gives up raises a CTA-wide
flag, all roles leave through the common exit (copies in flight are awaited, tensor memory is freed) and
the device status word records the time-out.  Nothing here faults, traps or hangs: the test shortens the
limit to about a millisecond and has the forward kernel's loader leave out one K-tile request (the
library's test aid), so that the wait for that tile expires by itself.
"""
import time

import numpy as np
import pytest
import torch

from paper_2608_00029_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["tiny", "tiny_d128"])
def test_forward_wait_runs_out_and_the_library_recovers(name):
    import oracle
    from paper_2608_00029_b200 import nova_attn as na
    dev = torch.device("cuda:0")
    cfg = W.CONFIGS["tiny"] if name == "tiny" else W.AttnConfig("tiny_d128", B=1, H=2, T=200, D=128, seed=5)
    Q, K, V, dO = W.make_inputs(cfg)
    q, k, v = (x.to(dev) for x in (Q, K, V))
    o = torch.zeros_like(q)
    lse = torch.zeros((cfg.B, cfg.H, cfg.T), dtype=torch.float32, device=dev)
    na.nova_attn_fwd(q, k, v, o, lse, cfg.scale, True)       # a normal call first: everything is set up
    na.nova_attn_poll_device_status()
    try:
        na.nova_attn_test_configure_waits(1 << 21, 1)         # about one millisecond; one K tile never requested
        t0 = time.perf_counter()
        na.nova_attn_fwd(q, k, v, o, lse, cfg.scale, True)
        with pytest.raises(na.NovaAttnError) as ei:
            na.nova_attn_poll_device_status()
        elapsed = time.perf_counter() - t0
        assert ei.value.status == na.ERR_TIMEOUT
        assert elapsed < 1.0, f"the kernel took {elapsed:.2f} s to give up"
    finally:
        na.nova_attn_test_configure_waits(0, 0)
    assert na.nova_attn_poll_device_status() == 0             # the poll cleared the status word
    # the same process, the same buffers: an ordinary call is correct again
    na.nova_attn_fwd(q, k, v, o, lse, cfg.scale, True)
    na.nova_attn_poll_device_status()
    O_ref, LSE_ref = oracle.attn_fwd(W.widen(Q), W.widen(K), W.widen(V), cfg.scale, True)
    assert (np.abs(W.widen(o) - O_ref) <= 1e-2 + 1e-2 * np.abs(O_ref)).all()
    assert (np.abs(W.widen(lse) - LSE_ref) <= 1e-2 + 1e-2 * np.abs(LSE_ref)).all()


def test_configure_waits_rejects_bad_arguments():
    from paper_2608_00029_b200 import nova_attn as na
    with pytest.raises(na.NovaAttnError):
        na.nova_attn_test_configure_waits(-5, 0)
    with pytest.raises(na.NovaAttnError):
        na.nova_attn_test_configure_waits(0, 7)
    na.nova_attn_test_configure_waits(0, 0)
