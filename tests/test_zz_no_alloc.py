"""tlr_route_static: the entry point for callers that may not allocate GPU memory.

It needs no context and uses a fixed scratch array inside the library.  Checked here
against the regular context-based entry point on the same inputs and against the CPU
oracle, for two calls in a row (the second with other inputs and fewer rows, so
leftovers of the first call in the shared scratch would show), and for the property it
exists for: the free device memory is the same before and after a call.  Collected last
on purpose: a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

import tlr_synth as S
from oracle import route_oracle as O
from tests.parity import ABS_TOL, REL_TOL, check_against_oracle, check_self_consistency, run_gpu

pytestmark = pytest.mark.gpu


def route_static(P, Wd, h_cpu, tau, with_status=True):
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
    h_dev = h_cpu.cuda()
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    P.tlr_route_static(d, V, Wd, h_dev, n, tau, token, conf, ent, mask, idx, cnt, status if with_status else None)
    torch.cuda.synchronize()
    free_after = torch.cuda.mem_get_info()[0]
    return {"token": token.cpu().numpy(), "conf": conf.cpu().numpy(), "entropy": ent.cpu().numpy(),
            "route_mask": mask.cpu().numpy(), "routed_idx": idx.cpu().numpy(), "routed_count": int(cnt.item()),
            "status": int(status.item()) if with_status else 0, "free_before": free_before, "free_after": free_after}


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
    W64 = O.bf16_bits_to_f64(S.bf16_bits(W))
    for call, (hid, tau) in enumerate(((first, 0.5), (second, 0.5))):
        got = route_static(pkg, Wd, hid.h, tau)
        want = run_gpu(pkg, Wd, hid.h, tau)
        assert got["status"] == 0 and want["status"] == 0
        assert 0 < want["routed_count"] < hid.h.shape[0]
        assert_same(got, want)
        # ... and against the oracle, like every other entry point
        ref = O.route_oracle(S.bf16_bits(hid.h), S.bf16_bits(W), tau, W64=W64)
        check_self_consistency(got, tau, V)
        rep = check_against_oracle(ref, got, O.bf16_bits_to_f64(S.bf16_bits(hid.h)), W64)
        if rep["route_exempt_rows"] == 0:
            assert got["routed_count"] == ref.routed_count
            assert np.array_equal(got["routed_idx"][:ref.routed_count], ref.routed_idx)
        if call > 0:      # past the one-time set-up: the call itself takes no device memory
            assert got["free_after"] == got["free_before"]


def test_static_entry_point_small_batch_and_no_status_word(pkg):
    # at most 64 rows takes the M = 64 form of the projection kernel; status_dev may be NULL
    d, V = 128, 9001
    W = S.make_W(d, V, seed=5, std=0.1)
    Wd = W.cuda()
    hid = S.make_h(16, d, seed=5, W=W, planted_fraction=0.25)
    ref = O.route_oracle(S.bf16_bits(hid.h), S.bf16_bits(W), 0.5)
    for with_status in (True, False):
        got = route_static(pkg, Wd, hid.h, 0.5, with_status=with_status)
        assert got["status"] == 0
        check_self_consistency(got, 0.5, V)
        check_against_oracle(ref, got)
        if not with_status:   # second call of this shape: kernels loaded, set-up done
            assert got["free_after"] == got["free_before"]


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
