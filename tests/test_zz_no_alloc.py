"""tlr_route_static: the entry point for callers that may not allocate GPU memory.

It needs no context and uses a fixed scratch array inside the library.  Checked here
against the regular context-based entry point on the same inputs, for two calls in a
row (the second with other inputs and fewer rows, so leftovers of the first call in
the shared scratch would show).  Collected last on purpose: a run that stops at the
first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

import tlr_synth as S
from tests.parity import ABS_TOL, REL_TOL, run_gpu

pytestmark = pytest.mark.gpu


def route_static(P, Wd, h_cpu, tau):
    n, d = h_cpu.shape
    V = Wd.shape[0]
    dev = Wd.device
    token = torch.full((n,), -7, dtype=torch.int32, device=dev)
    conf = torch.full((n,), float("nan"), device=dev)
    ent = torch.full((n,), float("nan"), device=dev)
    mask = torch.full((n,), 9, dtype=torch.uint8, device=dev)
    idx = torch.full((n,), -3, dtype=torch.int32, device=dev)
    cnt = torch.full((1,), -5, dtype=torch.int32, device=dev)
    status = torch.full((1,), 77, dtype=torch.int32, device=dev)
    P.tlr_route_static(d, V, Wd, h_cpu.cuda(), n, tau, token, conf, ent, mask, idx, cnt, status)
    torch.cuda.synchronize()
    return {"token": token.cpu().numpy(), "conf": conf.cpu().numpy(), "entropy": ent.cpu().numpy(),
            "route_mask": mask.cpu().numpy(), "routed_idx": idx.cpu().numpy(), "routed_count": int(cnt.item()),
            "status": int(status.item())}


def assert_same(a, b):
    assert np.array_equal(a["token"], b["token"])
    assert np.array_equal(a["route_mask"], b["route_mask"])
    assert a["routed_count"] == b["routed_count"]
    c = a["routed_count"]
    assert np.array_equal(a["routed_idx"][:c], b["routed_idx"][:c])
    assert np.max(np.abs(a["conf"] - b["conf"]), initial=0.0) <= ABS_TOL
    assert np.max(np.abs(a["conf"] - b["conf"]) / b["conf"], initial=0.0) <= REL_TOL
    assert np.max(np.abs(a["entropy"] - b["entropy"]), initial=0.0) <= ABS_TOL


def test_static_entry_point_matches_context_entry_point_twice(pkg):
    d, V = 256, 30011
    W = S.make_W(d, V, seed=3, std=0.08)
    Wd = W.cuda()
    first = S.make_h(300, d, seed=1, W=W, planted_fraction=0.1)
    second = S.make_h(77, d, seed=2, W=W, planted_fraction=0.2)
    for hid, tau in ((first, 0.5), (second, 0.5)):
        got = route_static(pkg, Wd, hid.h, tau)
        want = run_gpu(pkg, Wd, hid.h, tau)
        assert got["status"] == 0 and want["status"] == 0
        assert 0 < want["routed_count"] < hid.h.shape[0]
        assert_same(got, want)


def test_static_entry_point_small_hidden_size_and_limits(pkg):
    # d % 8 != 0 takes the CUDA-core kernel; more rows than the fixed scratch holds is an error
    W = S.make_W(36, 1500, seed=4, std=0.2)
    Wd = W.cuda()
    hid = S.make_h(20, 36, seed=4)
    assert_same(route_static(pkg, Wd, hid.h, 0.01), run_gpu(pkg, Wd, hid.h, 0.01))
    big = torch.zeros((pkg.TLR_STATIC_MAX_ROWS + 1, 36), dtype=torch.bfloat16)
    with pytest.raises(pkg.TlrError) as e:
        route_static(pkg, Wd, big, 0.5)
    assert e.value.code == 6
    empty = route_static(pkg, Wd, hid.h[:0], 0.5)
    assert empty["routed_count"] == 0
