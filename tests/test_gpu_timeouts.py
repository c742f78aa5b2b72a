"""Failure reporting of the prefetch-ring kernels, exercised without anything going wrong on
the device: the poll limit of their waits is set to zero, so every wait on a bulk asynchronous
copy gives up at once although the copy is on its way.  The kernels must then leave in order
(all threads of a block together, after the copies in flight have landed), report through the
device status word, and leave the device usable; the context must refuse further iterations."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2111_00705_b200 import binding as cd
from paper_2111_00705_b200 import synth

pytestmark = pytest.mark.gpu


def healthy_run(d=6 * 16384 + 100, n=2):
    """A fresh context on the same device still computes what the oracle computes."""
    g = torch.Generator(device="cuda").manual_seed(3)
    grads = torch.randn(n * d, generator=g, device="cuda")
    c = cd.CDAdam(d, n, cd.SIGN)
    c.set_tile(16384)
    o = orc.Oracle(d, n, orc.SIGN)
    for _ in range(2):
        c.step(grads)
        o.step(grads.cpu().numpy())
    c.device_status()
    assert np.array_equal(c.get_state("x").cpu().numpy(), o.state("x"))
    assert np.array_equal(c.get_state("ghat_w").cpu().numpy(), o.state("ghat_w"))
    c.close(); o.close()


def test_scaled_sign_ring_reports_a_wait_that_ran_out_and_the_device_stays_usable():
    d, n = 6 * 16384 + 100, 2
    grads = torch.randn(n * d, device="cuda")
    c = cd.CDAdam(d, n, cd.SIGN)
    c.set_tile(16384)                         # the worker kernel with the prefetch ring
    c.step(grads)
    c.device_status()                         # an ordinary iteration reports nothing
    c.set_wait_limit(0)
    c.step(grads)
    with pytest.raises(cd.CdadamError) as e:
        c.device_status()
    assert e.value.code == cd.ERR_TIMEOUT
    with pytest.raises(cd.CdadamError) as e:  # the state is void: no further iterations
        c.step(grads)
    assert e.value.code == cd.ERR_STATE
    c.close()
    healthy_run()


def test_topk_ring_reports_a_wait_that_ran_out_and_the_device_stays_usable():
    w = synth.workload("C3", scale=0.01, steps=3)       # d = 256,000: 62 whole tiles per row
    c = cd.CDAdam(w.d, w.n, cd.TOPK, k=w.k)
    c.set_tile(16384)                         # the dense pass with the prefetch ring
    c.step(w.grads(1, "cuda").reshape(-1))    # no threshold guess yet: the ring does not run
    c.step(w.grads(2, "cuda").reshape(-1))
    c.device_status()
    c.set_wait_limit(0)
    c.step(w.grads(3, "cuda").reshape(-1))
    with pytest.raises(cd.CdadamError) as e:
        c.device_status()
    assert e.value.code == cd.ERR_TIMEOUT
    with pytest.raises(cd.CdadamError) as e:
        c.step(w.grads(3, "cuda").reshape(-1))
    assert e.value.code == cd.ERR_STATE
    c.close()
    healthy_run()


def test_default_limit_is_restored_by_a_negative_value():
    d, n = 4 * 16384, 2
    grads = torch.randn(n * d, device="cuda")
    c = cd.CDAdam(d, n, cd.SIGN)
    c.set_tile(16384)
    c.set_wait_limit(0)
    c.set_wait_limit(-1)
    c.step(grads)
    c.device_status()
    c.close()
