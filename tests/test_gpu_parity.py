"""GPU parity: the CUDA path, called through the C-ABI, against the CPU fp64 oracle."""
import math

import numpy as np
import pytest
import torch

import tlr_synth as S
from oracle import route_oracle as O
from tests.parity import check_against_oracle, check_self_consistency, run_gpu

pytestmark = pytest.mark.gpu


def small_case(n, d, V, seed, std=0.1, planted=0.0):
    W = S.make_W(d, V, seed=seed, std=std)
    hid = S.make_h(n, d, seed=seed, W=W, planted_fraction=planted)
    return W, hid


PATHS = [pytest.param(1, id="simt"), pytest.param(2, id="tc")]

# sizes that span several row units, vocabulary tiles and chunks, with ragged tails
SMALL_SHAPES = [
    (1, 64, 300), (16, 64, 1000), (37, 128, 4099), (130, 72, 5000), (257, 896, 3001),
    (300, 200, 20011), (129, 1536, 2500), (64, 2048, 777), (513, 64, 70000),
    (64, 128, 3000), (65, 128, 3000), (49, 264, 1111),      # either side of the 64-row switch of the MMA's M
]


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("n,d,V", SMALL_SHAPES)
def test_small_elementwise(pkg, path, n, d, V):
    W, hid = small_case(n, d, V, seed=n + V, std=0.1, planted=0.1 if n >= 16 else 0.0)
    first = O.route_oracle(S.bf16_bits(hid.h), S.bf16_bits(W), 0.5)
    tau = O.percentile_tau(first.conf, 0.5) if n > 1 else 0.5     # half of the rows route
    ref = O.route_oracle(S.bf16_bits(hid.h), S.bf16_bits(W), tau)
    gpu = run_gpu(pkg, W.cuda(), hid.h, tau, path=path)
    assert gpu["status"] == 0
    assert gpu["plan"].path == path
    check_self_consistency(gpu, tau, V)
    h64 = O.bf16_bits_to_f64(S.bf16_bits(hid.h)); W64 = O.bf16_bits_to_f64(S.bf16_bits(W))
    rep = check_against_oracle(ref, gpu, h64, W64)
    if rep["route_exempt_rows"] == 0:
        assert gpu["routed_count"] == ref.routed_count
        assert np.array_equal(gpu["routed_idx"][:ref.routed_count], ref.routed_idx)
    assert 0 < ref.routed_count < n or n == 1      # the case exercises both outcomes


def test_hidden_size_not_multiple_of_8_uses_simt(pkg):
    W, hid = small_case(20, 36, 1500, seed=4)
    ref = O.route_oracle(S.bf16_bits(hid.h), S.bf16_bits(W), 0.01)
    gpu = run_gpu(pkg, W.cuda(), hid.h, 0.01)
    assert gpu["plan"].path == 1 and gpu["status"] == 0
    check_against_oracle(ref, gpu)
    check_self_consistency(gpu, 0.01, 1500)


@pytest.mark.parametrize("path", PATHS)
def test_empty_batch(pkg, path):
    W, hid = small_case(4, 64, 500, seed=1)
    gpu = run_gpu(pkg, W.cuda(), hid.h[:0], 0.5, path=path, max_n=4)
    assert gpu["routed_count"] == 0 and gpu["status"] == 0


@pytest.mark.parametrize("path", PATHS)
def test_threshold_extremes_and_monotone(pkg, path):
    W, hid = small_case(200, 128, 3000, seed=9, std=0.15, planted=0.2)
    Wd = W.cuda()
    prev = -1
    for tau in (0.0, 0.001, 0.01, 0.5, 0.999, 1.0):
        gpu = run_gpu(pkg, Wd, hid.h, tau, path=path)
        check_self_consistency(gpu, tau, 3000)
        assert gpu["routed_count"] >= prev
        prev = gpu["routed_count"]
        if tau == 0.0:
            assert gpu["routed_count"] == 0          # "small_only": nothing is routed
        if tau == 1.0:
            assert gpu["routed_count"] == 200 and np.array_equal(gpu["routed_idx"], np.arange(200))


@pytest.mark.parametrize("path", PATHS)
def test_threshold_equal_to_a_confidence_is_strict(pkg, path):
    W, hid = small_case(64, 64, 2000, seed=12, std=0.2)
    Wd = W.cuda()
    first = run_gpu(pkg, Wd, hid.h, 0.5, path=path)
    tau = float(np.sort(first["conf"])[20])             # exactly one row's fp32 confidence
    gpu = run_gpu(pkg, Wd, hid.h, tau, path=path)
    assert np.array_equal(gpu["conf"], first["conf"])    # deterministic
    assert gpu["routed_count"] == int((first["conf"] < np.float32(tau)).sum())
    assert gpu["route_mask"][np.argsort(first["conf"], kind="stable")[20]] == 0   # equal is not below


@pytest.mark.parametrize("path", PATHS)
def test_all_equal_logits(pkg, path):
    V, d = 5000, 64
    W = S.make_W(d, V, seed=2)
    h = torch.zeros((40, d), dtype=torch.bfloat16)
    gpu = run_gpu(pkg, W.cuda(), h, 0.5, path=path)
    assert np.all(gpu["token"] == 0)
    np.testing.assert_allclose(gpu["conf"], 1.0 / V, rtol=1e-5)
    np.testing.assert_allclose(gpu["entropy"], math.log(V), atol=1e-4)
    assert gpu["routed_count"] == 40


@pytest.mark.parametrize("path", PATHS)
def test_exact_ties_go_to_lowest_index(pkg, path):
    d, V, n = 64, 4000, 50
    W, hid = small_case(n, d, V, seed=21, std=0.3)
    ref = O.route_oracle(S.bf16_bits(hid.h), S.bf16_bits(W), 0.5)
    W2 = W.clone()
    # copy each row's winning embedding to a LOWER and a HIGHER index, far apart (other tiles / chunks)
    winners = np.unique(ref.token)
    lower = {}
    for k, v in enumerate(winners.tolist()):
        lo, hi = k, V - 1 - k
        if lo < v:
            W2[lo] = W[v]; lower[v] = lo
        if hi > v:
            W2[hi] = W[v]
    ref2 = O.route_oracle(S.bf16_bits(hid.h), S.bf16_bits(W2), 0.5)
    gpu = run_gpu(pkg, W2.cuda(), hid.h, 0.5, path=path)
    clear = ref2.top2_gap == 0.0          # rows whose maximum is now duplicated exactly
    assert clear.sum() > n // 2
    assert np.array_equal(gpu["token"][clear], ref2.token[clear])


@pytest.mark.parametrize("path", PATHS)
def test_winner_in_last_vocabulary_row_and_at_boundaries(pkg, path):
    d, V = 128, 151936 // 8 + 5            # 18997: not a multiple of 16
    W = S.make_W(d, V, seed=5)
    targets = [V - 1, V - 2, 0, 15, 16, 255, 256, 257, 1023, 1024, 4095, 4096, V // 2, V - 17]
    g = torch.randn((len(targets), d), generator=torch.Generator().manual_seed(1), dtype=torch.float32).double()
    w = W[torch.tensor(targets)].double()
    g = g + 8.0 * w / w.pow(2).mean(dim=1, keepdim=True).sqrt()
    h = (g / g.pow(2).mean(dim=1, keepdim=True).sqrt() * 4.0).to(torch.bfloat16)
    ref = O.route_oracle(S.bf16_bits(h), S.bf16_bits(W), 0.5)
    assert ref.token.tolist() == targets
    gpu = run_gpu(pkg, W.cuda(), h, 0.5, path=path)
    assert gpu["token"].tolist() == targets
    check_against_oracle(ref, gpu)


def test_non_finite_row_is_routed_and_flagged(pkg):
    W, hid = small_case(8, 64, 1000, seed=3)
    h = hid.h.clone()
    h[3, 5] = float("nan")
    gpu = run_gpu(pkg, W.cuda(), h, 0.0)
    assert gpu["route_mask"].tolist() == [0, 0, 0, 1, 0, 0, 0, 0]
    assert gpu["routed_idx"][:1].tolist() == [3] and gpu["routed_count"] == 1
    assert gpu["status"] & pkg.TLR_DEV_NONFINITE


def test_two_runs_bit_identical_and_paths_agree(pkg):
    W, hid = small_case(300, 256, 30000, seed=17, planted=0.05)
    Wd = W.cuda()
    a = run_gpu(pkg, Wd, hid.h, 0.5, path=2)
    b = run_gpu(pkg, Wd, hid.h, 0.5, path=2)
    for k in ("token", "conf", "entropy", "route_mask"):
        assert np.array_equal(a[k], b[k]), k
    c = run_gpu(pkg, Wd, hid.h, 0.5, path=1)
    assert np.array_equal(a["route_mask"], c["route_mask"])
    np.testing.assert_allclose(a["conf"], c["conf"], rtol=1e-3)


@pytest.mark.parametrize("how,n,d,V", [("pinned", 100, 128, 6000),      # h fetched by the copy kernel
                                       ("pageable", 100, 128, 6000),    # h through the copy engine
                                       ("pinned", 300, 896, 3001),      # pair kernel behind the copy kernel
                                       ("pinned", 2500, 896, 2048),     # more than 4 MB of h: copy engine again
                                       ("pinned", 37, 64, 999),         # odd max_n: the status word's alignment
                                       ("pinned", 0, 128, 6000)])
def test_host_buffer_entry_point(pkg, how, n, d, V):
    W, hid = small_case(max(n, 1), d, V, seed=6, planted=0.1)
    hrows = hid.h[:n]
    Wd = W.cuda()
    ctx = pkg.tlr_create(d, V, Wd, max(n, 1) + 28)
    pin = (lambda x: x.pin_memory()) if how == "pinned" else (lambda x: x)
    h = pin(hrows.contiguous())
    m = max(n, 1)
    token = pin(torch.empty(m, dtype=torch.int32)); conf = pin(torch.empty(m))
    ent = pin(torch.empty(m)); mask = pin(torch.empty(m, dtype=torch.uint8))
    idx = pin(torch.full((m,), -1, dtype=torch.int32)); cnt = pin(torch.full((1,), -9, dtype=torch.int32))
    for _ in range(2):                                  # twice: the context's staging is reused
        pkg.tlr_route_host(ctx, h, n, 0.5, token, conf, ent, mask, idx, cnt)
    if n == 0:
        assert int(cnt.item()) == 0
        pkg.tlr_destroy(ctx)
        return
    ref = O.route_oracle(S.bf16_bits(hrows), S.bf16_bits(W), 0.5)
    gpu = {"token": token.numpy()[:n], "conf": conf.numpy()[:n], "entropy": ent.numpy()[:n],
           "route_mask": mask.numpy()[:n], "routed_idx": idx.numpy(), "routed_count": int(cnt.item())}
    rep = check_against_oracle(ref, gpu)
    check_self_consistency(gpu, 0.5, V)
    if rep["route_exempt_rows"] == 0:
        assert gpu["routed_count"] == ref.routed_count
    assert pkg.tlr_last_device_status(ctx) == 0
    pkg.tlr_destroy(ctx)


def test_two_host_calls_in_flight(pkg):
    """submit / collect: batches of different sizes are handed in while earlier ones are still on the GPU; every
    collect returns the oldest call's results, which must be the oracle's for THAT batch."""
    d, V = 256, 9001
    W, _ = small_case(8, d, V, seed=12, planted=0.0)
    Wd = W.cuda()
    sizes = [300, 40, 129, 1, 300, 0, 64]                 # pair kernel, one-CTA kernels, an empty batch
    batches = [S.make_h(n, d, seed=20 + i, W=W, planted_fraction=0.2 if n >= 5 else 0.0).h.pin_memory()
               for i, n in enumerate(sizes)]
    refs = [O.route_oracle(S.bf16_bits(b), S.bf16_bits(W), 0.5) if b.shape[0] else None for b in batches]
    ctx = pkg.tlr_create(d, V, Wd, max(sizes))
    m = max(sizes)
    outs = lambda: (torch.empty(m, dtype=torch.int32).pin_memory(), torch.empty(m).pin_memory(), torch.empty(m).pin_memory(),
                    torch.empty(m, dtype=torch.uint8).pin_memory(), torch.full((m,), -1, dtype=torch.int32).pin_memory(),
                    torch.full((1,), -9, dtype=torch.int32).pin_memory())

    def check(i, o):
        n = sizes[i]
        if n == 0:
            assert int(o[5].item()) == 0
            return
        gpu = {"token": o[0].numpy()[:n], "conf": o[1].numpy()[:n], "entropy": o[2].numpy()[:n],
               "route_mask": o[3].numpy()[:n], "routed_idx": o[4].numpy(), "routed_count": int(o[5].item())}
        rep = check_against_oracle(refs[i], gpu)
        check_self_consistency(gpu, 0.5, V)
        if rep["route_exempt_rows"] == 0:
            assert gpu["routed_count"] == refs[i].routed_count
            assert np.array_equal(gpu["routed_idx"][:refs[i].routed_count], refs[i].routed_idx)

    pkg.tlr_route_host_submit(ctx, batches[0], sizes[0], 0.5)
    for i in range(1, len(sizes)):
        pkg.tlr_route_host_submit(ctx, batches[i], sizes[i], 0.5)          # two in flight now
        with pytest.raises(pkg.TlrError) as e:
            pkg.tlr_route_host_submit(ctx, batches[i], sizes[i], 0.5)      # a third is refused
        assert e.value.code == 1
        o = outs()
        pkg.tlr_route_host_collect(ctx, *o)
        check(i - 1, o)
    with pytest.raises(pkg.TlrError):                                      # the one-call form is refused meanwhile
        pkg.tlr_route_host(ctx, batches[0], sizes[0], 0.5, *outs())
    o = outs()
    pkg.tlr_route_host_collect(ctx, *o)
    check(len(sizes) - 1, o)
    with pytest.raises(pkg.TlrError) as e:
        pkg.tlr_route_host_collect(ctx, *outs())                           # nothing left to collect
    assert e.value.code == 1
    o = outs()
    pkg.tlr_route_host(ctx, batches[2], sizes[2], 0.5, *o)                 # and the one-call form works again
    check(2, o)
    assert pkg.tlr_last_device_status(ctx) == 0
    pkg.tlr_destroy(ctx)


def test_argument_errors(pkg):
    W, hid = small_case(4, 64, 500, seed=1)
    Wd = W.cuda()
    L = pkg.load_library()
    import ctypes
    ctx = ctypes.c_void_p(0)
    assert L.tlr_create(0, 500, ctypes.c_void_p(Wd.data_ptr()), 4, ctypes.byref(ctx)) == 1
    assert L.tlr_create(64, 500, ctypes.c_void_p(0), 4, ctypes.byref(ctx)) == 1
    assert L.tlr_create(64, 500, ctypes.c_void_p(Wd.data_ptr() + 2), 4, ctypes.byref(ctx)) == 2
    router = pkg.Router(Wd, max_n=4)
    with pytest.raises(pkg.TlrError) as e:
        pkg.tlr_route(router.ctx, hid.h.cuda(), 5, 0.5, router.token, router.conf, router.entropy,
                      router.route_mask, router.routed_idx, router.routed_count)
    assert e.value.code == 6
    with pytest.raises(pkg.TlrError) as e:
        pkg.tlr_route(router.ctx, None, 4, 0.5, router.token, router.conf, router.entropy,
                      router.route_mask, router.routed_idx, router.routed_count)
    assert e.value.code == 1
    with pytest.raises(pkg.TlrError) as e:
        pkg.tlr_route(router.ctx, hid.h.cuda().data_ptr() + 2, 3, 0.5, router.token, router.conf, router.entropy,
                      router.route_mask, router.routed_idx, router.routed_count)
    assert e.value.code == 2
    router.close()


@pytest.mark.parametrize("path", PATHS)
def test_degenerate_vocabulary_and_tiny_shapes(pkg, path):
    # V = 1: the only token has probability 1, entropy 0, and is never "below" any tau <= 1
    W = S.make_W(8, 1, seed=1, std=0.5)
    hid = S.make_h(5, 8, seed=1)
    gpu = run_gpu(pkg, W.cuda(), hid.h, 1.0, path=path)
    assert gpu["token"].tolist() == [0] * 5 and np.all(np.abs(gpu["conf"] - 1.0) < 1e-6) and np.all(gpu["entropy"] < 1e-6)
    assert gpu["routed_count"] == 0
    # V = 17 (one row past a 16-row granule), d = 16; and d = 8 with n past one row unit
    for n, d, V in ((5, 16, 17), (200, 8, 33), (129, 8, 16)):
        W = S.make_W(d, V, seed=V, std=0.7)
        hid = S.make_h(n, d, seed=n)
        ref = O.route_oracle(S.bf16_bits(hid.h), S.bf16_bits(W), 0.3)
        gpu = run_gpu(pkg, W.cuda(), hid.h, 0.3, path=path)
        assert gpu["status"] == 0
        check_self_consistency(gpu, 0.3, V)
        check_against_oracle(ref, gpu, O.bf16_bits_to_f64(S.bf16_bits(hid.h)), O.bf16_bits_to_f64(S.bf16_bits(W)))


def test_prepared_call_is_the_same_step(pkg):
    """Router.prepared marshals the arguments once; calling it is bit-identical to route()."""
    W, hid = small_case(150, 128, 6000, seed=21, planted=0.1)
    r = pkg.Router(W.cuda(), max_n=150)
    h = hid.h.cuda()
    r.route(h, 0.4)
    torch.cuda.synchronize()
    want = [t.clone() for t in (r.token, r.conf, r.entropy, r.route_mask, r.routed_count)]
    want_idx = r.routed_idx[:int(r.routed_count.item())].clone()
    call = r.prepared(h, 0.4)
    for _ in range(3):
        r.token.fill_(-1); r.routed_count.fill_(-1)
        call()
    torch.cuda.synchronize()
    for got, w in zip((r.token, r.conf, r.entropy, r.route_mask, r.routed_count), want):
        assert torch.equal(got, w)
    assert torch.equal(r.routed_idx[:int(r.routed_count.item())], want_idx)
    with pytest.raises(ValueError):
        r.prepared(h.float(), 0.4)
    r.close()
