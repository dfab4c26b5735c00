"""tlr_route inside a CUDA graph: the call allocates nothing, reads nothing back and does not synchronise, so a
decode loop can capture it once and replay it.  The replayed results must equal the eagerly launched ones bit for
bit, for the one-CTA kernel, the CTA-pair kernel and the 8-bit head, and follow the input buffer's new contents."""
import numpy as np
import pytest
import torch

import tlr_synth as S
from tests.parity import to_np

pytestmark = pytest.mark.gpu


def snapshot(r, n):
    return (to_np(r.token[:n]).copy(), to_np(r.conf[:n]).copy(), to_np(r.entropy[:n]).copy(),
            to_np(r.route_mask[:n]).copy(), int(r.routed_count.item()))


@pytest.mark.parametrize("n,fp8", [(16, False), (100, False), (300, False), (16, True)])
def test_capture_and_replay(pkg, n, fp8):
    d, V = 256, 9000
    if fp8:
        codes, scale = S.make_W8(d, V, seed=4, std=0.1)
        r = pkg.Router(codes.cuda(), max_n=n, wscale=scale.cuda())
    else:
        r = pkg.Router(S.make_W(d, V, seed=4, std=0.1).cuda(), max_n=n)
    h_a = S.make_h(n, d, seed=1).h.cuda()
    h_b = S.make_h(n, d, seed=2).h.cuda()
    buf = h_a.clone()

    r.route(buf, 0.01)                                   # eager, input A
    torch.cuda.synchronize()
    eager_a = snapshot(r, n)
    buf.copy_(h_b)
    r.route(buf, 0.01)                                   # eager, input B
    torch.cuda.synchronize()
    eager_b = snapshot(r, n)
    assert not np.array_equal(eager_a[1], eager_b[1])

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    buf.copy_(h_a)
    torch.cuda.synchronize()
    with torch.cuda.graph(g, stream=side):
        r.route(buf, 0.01)
    for want, src in ((eager_a, h_a), (eager_b, h_b), (eager_a, h_a)):
        buf.copy_(src)
        r.token.fill_(-1); r.conf.fill_(float("nan"))
        g.replay()
        torch.cuda.synchronize()
        got = snapshot(r, n)
        for a, b in zip(want, got):
            assert np.array_equal(a, b)
    assert pkg.tlr_last_device_status(r.ctx) == 0
    del g
    r.close()
