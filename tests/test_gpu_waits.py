"""Device-side waits that run out: every kernel of the library that waits for another party does so for a
bounded time.  rad_wait_probe runs the very wait helpers of those kernels on something that is never
signalled, in tiny kernels that hold no tensor memory and have no copy in flight, so the wait expires: the
kernel must return, report RAD_DEV_ETIMEOUT and leave the context and the stream usable.  Nothing here
faults, traps or hangs; the longest wait is 2 ms."""
import time

import numpy as np
import pytest
import torch

from oracle import rad as orc
from workloads import layer_inputs

from gpu_util import bits_host, to_dev, u32
from layout import bits_of, tile_major

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("which", ["pair_barrier", "pipe_barrier", "lookback"])
def test_a_wait_that_nothing_ends_gives_up_and_the_next_call_is_exact(which):
    import paper_2007_10412_b200 as rad
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    rad.rad_wait_probe(which, 2_000_000, status)          # 2 ms
    torch.cuda.synchronize()                              # the kernel returned
    waited = time.perf_counter() - t0
    assert status.item() == rad.RAD_DEV_ETIMEOUT
    assert 0.0015 < waited < 1.0
    # the status word is sticky: a second code does not overwrite the first
    rad.rad_wait_probe(which, 1_000_000, status)
    torch.cuda.synchronize()
    assert status.item() == rad.RAD_DEV_ETIMEOUT
    # an ordinary call on the same stream right after it: bit for bit the oracle's store
    B, D, p = 700, 1160, 0.1
    A, _ = layer_inputs(B, D, 1, dtype="bf16", seed=9, relu_like=True)
    ref = orc.forward_store(A, "bf16", "different", p, 5, 1, 2)
    prev = rad.rad_set_store_kernel("pipelined")
    try:
        st = rad.Store("different", "bf16", B, D, p, seed=5, layer=1, step=2)
        ok = torch.zeros(1, dtype=torch.int32, device="cuda")
        rad.rad_linear_forward_store(to_dev(A, "bf16"), st, ok)
        torch.cuda.synchronize()
    finally:
        rad.rad_set_store_kernel(prev)
    assert ok.item() == 0
    kb, vals, offs = tile_major(ref)
    assert np.array_equal(u32(st.keepbits), kb) and np.array_equal(u32(st.offsets), offs)
    assert np.array_equal(bits_host(st.values[:int(offs[-1])]), bits_of(vals, "bf16"))


def test_wait_limit_setting_and_argument_checks():
    import paper_2007_10412_b200 as rad
    prev = rad.rad_set_wait_limit_ns(0)
    assert prev == 2_000_000_000                          # the default: 2 s
    assert rad.rad_set_wait_limit_ns(500_000_000) == prev
    assert rad.rad_set_wait_limit_ns(prev) == 500_000_000
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(rad.RadError, match="invalid"):
        rad.rad_wait_probe("lookback", 5_000_000_000, status)      # probes wait a second at most
    with pytest.raises(rad.RadError, match="invalid"):
        rad.rad_wait_probe("lookback", 0, status)
