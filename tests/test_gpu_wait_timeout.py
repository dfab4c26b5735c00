"""Failure handling of the projection kernel, without faulting or hanging the GPU.

Every barrier wait in the kernel is bounded.  The test hook makes the W producer issue no
copies, so the consumers' waits run out; the kernel must then raise TLR_DEV_WAIT_TIMEOUT, return
by itself, and leave the context fully usable for the next call."""
import numpy as np
import pytest
import torch

import tlr_synth as S
from tests.parity import to_np

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n", [48, 300])          # one CTA per worker / a pair of CTAs per worker
def test_wait_runs_out_and_context_survives(pkg, n):
    d, V = 128, 40000
    W = S.make_W(d, V, seed=2, std=0.1)
    hid = S.make_h(n, d, seed=3)
    r = pkg.Router(W.cuda(), max_n=n)
    h = hid.h.cuda()

    def run():
        r.route(h, 0.01)
        torch.cuda.synchronize()
        return to_np(r.token[:n]).copy(), to_np(r.conf[:n]).copy(), int(r.routed_count.item())

    good = run()
    assert pkg.tlr_last_device_status(r.ctx) == 0

    pkg.tlr_debug_inject(r.ctx, 1, 200)             # copies dropped, every wait limited to 0.2 s
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record(); r.route(h, 0.01); t1.record()
    torch.cuda.synchronize()                        # returns: the kernel gave up by itself
    assert t0.elapsed_time(t1) < 5000.0
    assert pkg.tlr_last_device_status(r.ctx) & pkg.TLR_DEV_WAIT_TIMEOUT

    # the host-buffer entry point reports the condition as an error code
    pin = hid.h.pin_memory()
    cnt = torch.zeros(1, dtype=torch.int32).pin_memory()
    with pytest.raises(pkg.TlrError) as e:
        pkg.tlr_route_host(r.ctx, pin, n, 0.01, None, None, None, None, None, cnt)
    assert e.value.code == 7
    pkg.tlr_last_device_status(r.ctx)               # clear

    pkg.tlr_debug_inject(r.ctx, 0, 0)
    again = run()
    assert pkg.tlr_last_device_status(r.ctx) == 0
    assert np.array_equal(good[0], again[0]) and np.array_equal(good[1], again[1]) and good[2] == again[2]
    r.close()


def test_wait_runs_out_on_the_8bit_head(pkg):
    """The same hook on the fp8 decode kernel: the flag is raised, the kernel returns, the context recovers."""
    n, d, V = 24, 128, 40000
    codes, scale = S.make_W8(d, V, seed=2, std=0.1)
    r = pkg.Router(codes.cuda(), max_n=n, wscale=scale.cuda())
    h = S.make_h(n, d, seed=3).h.cuda()

    def run():
        r.route(h, 0.01)
        torch.cuda.synchronize()
        return to_np(r.token[:n]).copy(), to_np(r.conf[:n]).copy(), int(r.routed_count.item())

    good = run()
    assert pkg.tlr_last_device_status(r.ctx) == 0
    pkg.tlr_debug_inject(r.ctx, 1, 200)
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record(); r.route(h, 0.01); t1.record()
    torch.cuda.synchronize()
    assert t0.elapsed_time(t1) < 5000.0
    assert pkg.tlr_last_device_status(r.ctx) & pkg.TLR_DEV_WAIT_TIMEOUT
    pkg.tlr_debug_inject(r.ctx, 0, 0)
    again = run()
    assert pkg.tlr_last_device_status(r.ctx) == 0
    assert np.array_equal(good[0], again[0]) and np.array_equal(good[1], again[1]) and good[2] == again[2]
    r.close()
