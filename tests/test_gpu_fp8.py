"""The routing step on an 8-bit (e4m3, one scale per row) copy of W, for decode batches: the CUDA path
(tlr_create_fp8, called through the C-ABI) against the oracle run on the de-quantised matrix."""
import ctypes

import numpy as np
import pytest
import torch

import tlr_synth as S
from oracle import route_oracle as O
from tests.parity import check_against_oracle, check_self_consistency, to_np

pytestmark = pytest.mark.gpu


class FullHead8:
    """One full-size 8-bit head at a time: codes and scales on the host and the device, and the fp64 matrix
    they stand for (1-2 GB)."""
    key = None
    codes_dev = scale_dev = w64 = None
    host = None

    @classmethod
    def get(cls, d, V):
        if cls.key != (d, V):
            cls.codes_dev = cls.scale_dev = cls.w64 = cls.host = None
            codes, scale = S.make_W8(d, V, seed=0)
            cls.host = (codes, scale)
            cls.w64 = O.dequantize_e4m3(codes.numpy(), scale.numpy())
            cls.codes_dev, cls.scale_dev = codes.cuda(), scale.cuda()
            cls.key = (d, V)
        return cls.host


def run_fp8(P, codes, scale, h_cpu, tau, max_n=None, on_device=False, **kw):
    n = h_cpu.shape[0]
    r = P.Router(codes if on_device else codes.cuda(), max_n=max(1, max_n or n),
                 wscale=scale if on_device else scale.cuda())
    r.token.fill_(-7); r.conf.fill_(float("nan")); r.entropy.fill_(float("nan"))
    r.route_mask.fill_(9); r.routed_idx.fill_(-3); r.routed_count.fill_(-5)
    h = h_cpu.cuda() if n > 0 else torch.empty((0, codes.shape[1]), dtype=torch.bfloat16, device="cuda")
    r.route(h, tau, **kw)
    torch.cuda.synchronize()
    out = {"token": to_np(r.token[:n]), "conf": to_np(r.conf[:n]), "entropy": to_np(r.entropy[:n]),
           "route_mask": to_np(r.route_mask[:n]), "routed_idx": to_np(r.routed_idx),
           "routed_count": int(r.routed_count.item()), "status": P.tlr_last_device_status(r.ctx),
           "plan": P.tlr_plan_query(r.ctx, n)}
    r.close()
    return out


def planted_h(n, d, W64, seed):
    """Unit-RMS rows, a tenth of them pushed along a row of the de-quantised head (confident rows)."""
    hid = S.make_h(n, d, seed=seed)
    g = hid.h.double().numpy().copy()
    rng = np.random.default_rng(seed)
    for i in rng.choice(n, size=n // 10, replace=False) if n >= 10 else []:
        w = W64[rng.integers(0, W64.shape[0])]
        g[i] += 8.0 * w / np.sqrt((w * w).mean())
        g[i] /= np.sqrt((g[i] * g[i]).mean())
    return torch.from_numpy(g).to(torch.bfloat16)


# several tiles and chunks, ragged vocabulary tails, d not a multiple of the 128-wide slab, 1..128 rows (above 64
# rows the two parts of h take an MMA each)
SHAPES = [(16, 128, 1024), (5, 256, 3000), (64, 896, 20011), (33, 144, 777), (1, 64, 300), (48, 2048, 5000),
          (17, 16, 40), (65, 128, 3000), (100, 896, 20011), (128, 2048, 5000), (81, 272, 1500), (128, 64, 70000)]


@pytest.mark.parametrize("n,d,V", SHAPES)
def test_fp8_head_matches_oracle_on_dequantised_matrix(pkg, n, d, V):
    codes, scale = S.make_W8(d, V, seed=n + V, std=0.1)
    W64 = O.dequantize_e4m3(codes.numpy(), scale.numpy())
    h = planted_h(n, d, W64, seed=n + V)
    first = O.route_oracle(S.bf16_bits(h), None, 0.5, W64=W64)
    tau = O.percentile_tau(first.conf, 0.5) if n > 1 else 0.5
    ref = O.route_oracle(S.bf16_bits(h), None, tau, W64=W64)
    gpu = run_fp8(pkg, codes, scale, h, tau)
    assert gpu["status"] == 0
    assert gpu["plan"].launches == (2 if n <= 16 and d <= 1024 else 3)   # small batches of a small head: the kernel splits h itself
    check_self_consistency(gpu, tau, V)
    rep = check_against_oracle(ref, gpu, O.bf16_bits_to_f64(S.bf16_bits(h)), W64)
    if rep["route_exempt_rows"] == 0:
        assert gpu["routed_count"] == ref.routed_count
        assert np.array_equal(gpu["routed_idx"][:ref.routed_count], ref.routed_idx)


# The shapes the benchmark times with --fp8, in its launch configuration: the 0.5B-class head with 16 rows
# (the kernel splits h itself) and the d = 2048 head of the batch sweep with 1 and 64 rows (separate split kernel,
# shallower W ring).  Every row is compared with the oracle on the de-quantised matrix.
# Last: the 0.5B-class head with 128 rows, where every K step takes two MMAs (one per part of h).
FULL_SIZE = [("decode16", 16, True), ("sweep1", 1, False), ("sweep64", 64, False), ("decode16", 128, False)]


@pytest.mark.parametrize("name,n,inline", FULL_SIZE)
def test_fp8_head_at_benchmark_sizes(pkg, name, n, inline):
    wl = S.WORKLOADS[name]
    codes, scale = FullHead8.get(wl.d, wl.V)
    W64 = FullHead8.w64
    hid = S.make_h(n, wl.d, seed=0)
    first = O.route_oracle(S.bf16_bits(hid.h), None, 0.5, W64=W64)
    tau = O.percentile_tau(first.conf, 0.5) if n > 1 else 0.5
    ref = O.with_threshold(first, tau)
    gpu = run_fp8(pkg, FullHead8.codes_dev, FullHead8.scale_dev, hid.h, tau, on_device=True)
    assert gpu["status"] == 0
    assert gpu["plan"].launches == (2 if inline else 3)
    assert gpu["plan"].grid >= 140                       # the whole GPU streams W, as in the benchmark
    check_self_consistency(gpu, tau, wl.V)
    rep = check_against_oracle(ref, gpu, O.bf16_bits_to_f64(S.bf16_bits(hid.h)), W64)
    if rep["route_exempt_rows"] == 0:
        assert gpu["routed_count"] == ref.routed_count
        assert np.array_equal(gpu["routed_idx"][:ref.routed_count], ref.routed_idx)


def test_fp8_rows_with_a_wide_range_of_magnitudes(pkg):
    """Elements far below a row's largest (where the two-part split of h is no longer exact) and rows of very
    different scale: the result must stay within the usual tolerance."""
    n, d, V = 24, 256, 4000
    codes, scale = S.make_W8(d, V, seed=11, std=0.1)
    W64 = O.dequantize_e4m3(codes.numpy(), scale.numpy())
    g = S.make_h(n, d, seed=11).h.double()
    g[:, ::7] *= 2.0 ** -12                       # tiny elements beside ordinary ones
    g[3] *= 2.0 ** 10                              # one row much larger than the others ...
    g[4] *= 2.0 ** -10                             # ... one much smaller
    g[5] = 0.0                                     # and an all-zero row (uniform distribution)
    h = g.to(torch.bfloat16)
    ref = O.route_oracle(S.bf16_bits(h), None, 0.5, W64=W64)
    gpu = run_fp8(pkg, codes, scale, h, 0.5)
    assert gpu["status"] == 0
    check_against_oracle(ref, gpu, O.bf16_bits_to_f64(S.bf16_bits(h)), W64)
    assert gpu["conf"][5] == pytest.approx(1.0 / V, rel=1e-5) and gpu["token"][5] == 0


def test_fp8_empty_batch_options_and_host_buffers(pkg):
    n, d, V = 40, 128, 6000
    codes, scale = S.make_W8(d, V, seed=2, std=0.1)
    W64 = O.dequantize_e4m3(codes.numpy(), scale.numpy())
    h = planted_h(n, d, W64, seed=2)
    assert run_fp8(pkg, codes, scale, h[:0], 0.5, max_n=4)["routed_count"] == 0
    # per-row thresholds and the opposite polarity go through the same merge kernel
    ref = O.route_oracle(S.bf16_bits(h), None, 0.5, W64=W64)
    taus = torch.full((n,), 0.5)
    gpu = run_fp8(pkg, codes, scale, h, 0.0, tau_per_row=taus.cuda(), route_above=True)
    decided = np.abs(ref.conf - 0.5) > 1e-3 * 0.5
    assert np.array_equal(gpu["route_mask"][decided], (ref.conf > 0.5).astype(np.uint8)[decided])
    # host-buffer entry point
    ctx = pkg.tlr_create_fp8(d, V, codes.cuda(), scale.cuda(), n)
    tok = torch.empty(n, dtype=torch.int32).pin_memory(); conf = torch.empty(n).pin_memory(); ent = torch.empty(n).pin_memory()
    mask = torch.empty(n, dtype=torch.uint8).pin_memory(); idx = torch.empty(n, dtype=torch.int32).pin_memory()
    cnt = torch.zeros(1, dtype=torch.int32).pin_memory()
    pkg.tlr_route_host(ctx, h.pin_memory(), n, 0.5, tok, conf, ent, mask, idx, cnt)
    host = {"token": tok.numpy(), "conf": conf.numpy(), "entropy": ent.numpy(), "route_mask": mask.numpy(),
            "routed_idx": idx.numpy(), "routed_count": int(cnt.item())}
    check_against_oracle(ref, host, O.bf16_bits_to_f64(S.bf16_bits(h)), W64)
    pkg.tlr_destroy(ctx)


def test_fp8_argument_errors(pkg):
    codes, scale = S.make_W8(64, 500, seed=1)
    cd, sd = codes.cuda(), scale.cuda()
    L = pkg.load_library()
    ctx = ctypes.c_void_p(0)
    P = ctypes.c_void_p
    assert L.tlr_create_fp8(64, 500, P(0), P(sd.data_ptr()), 8, ctypes.byref(ctx)) == 1          # no W
    assert L.tlr_create_fp8(64, 500, P(cd.data_ptr()), P(0), 8, ctypes.byref(ctx)) == 1          # no scales
    assert L.tlr_create_fp8(64, 500, P(cd.data_ptr() + 1), P(sd.data_ptr()), 8, ctypes.byref(ctx)) == 2
    assert L.tlr_create_fp8(72, 400, P(cd.data_ptr()), P(sd.data_ptr()), 8, ctypes.byref(ctx)) == 3   # d % 16 != 0
    r = pkg.Router(cd, max_n=200, wscale=sd)
    h = torch.zeros((129, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(pkg.TlrError) as e:
        r.route(h, 0.5)
    assert e.value.code == 3                                                                         # more than 128 rows
    with pytest.raises(pkg.TlrError):
        pkg.tlr_set_path(r.ctx, pkg.TLR_PATH_SIMT)
    r.close()
