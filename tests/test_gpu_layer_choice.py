"""pact_key_spread against the oracle: the largest key distance of each layer and the earliest layer
that reaches a threshold (the layer choice described after Eq. 11)."""
import numpy as np
import pytest
import torch

from oracle import pact_oracle as orc
from paper_2504_08966_b200 import workloads
from tests.helpers import f64

pytestmark = pytest.mark.gpu


def _tolerance(d_k):
    # fp32 accumulation of d_k exact products plus two fp32 inverse norms and the final rounding
    return (d_k + 4) * 2.0 ** -24


def _run(layers, threshold, dtype, n_h, d_h):
    from paper_2504_08966_b200 import binding as pb
    ctx = pb.Context(64, n_h, n_h, d_h, dtype, torch.bfloat16)
    dev = [K.cuda() for K in layers]
    md = torch.full((len(layers),), -7.0, dtype=torch.float32, device="cuda")
    lo = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    ctx.pact_key_spread(dev, threshold, md, lo)
    torch.cuda.synchronize()
    return md.cpu().numpy().astype(np.float64), int(lo.item())


def _oracle(layers):
    return np.array([orc.max_key_distance(f64(K)) for K in layers])


def _thresholds(want):
    """Thresholds that sit well away from every layer's value, so that fp32 and fp64 agree."""
    s = np.sort(np.unique(want))
    mids = [(a + b) / 2 for a, b in zip(s[:-1], s[1:]) if b - a > 1e-3]
    return [0.0] + mids + [float(s[-1]) + 0.01, 2.5]


@pytest.mark.parametrize("N", [1, 2, 127, 129, 1000])
def test_spread_bf16_matches_oracle_across_tile_edges(N):
    layers = workloads.layer_keys(seed=11, n_layers=6, N=N, n_h=4, d_h=128)
    want = _oracle(layers)
    got, _ = _run(layers, 0.5, torch.bfloat16, 4, 128)
    assert np.abs(got - want).max() <= _tolerance(512)
    if N == 1:
        assert (got == 0).all()
    for t in _thresholds(want):
        _, layer = _run(layers, t, torch.bfloat16, 4, 128)
        assert layer == orc.select_layer([f64(K) for K in layers], t)


def test_spread_fp32_keys_and_more_layers_than_one_launch_takes():
    layers = workloads.layer_keys(seed=12, n_layers=37, N=150, n_h=2, d_h=64, dtype=torch.float32)
    want = _oracle(layers)
    got, _ = _run(layers, 0.5, torch.float32, 2, 64)
    assert np.abs(got - want).max() <= 2.0 ** -22          # double arithmetic, rounded to fp32 once
    for t in _thresholds(want):
        _, layer = _run(layers, t, torch.float32, 2, 64)
        assert layer == orc.select_layer([f64(K) for K in layers], t)
    # the qualifying layer sits in the third group of sixteen
    mix = [0.01] * 37
    mix[35] = 1.0
    late = workloads.layer_keys(seed=13, n_layers=37, N=150, n_h=2, d_h=64, dtype=torch.float32, mix=mix)
    got, layer = _run(late, 0.2, torch.float32, 2, 64)
    assert layer == 35 == orc.select_layer([f64(K) for K in late], 0.2)


def test_spread_bf16_keys_of_a_width_the_tensor_core_tiles_do_not_take():
    layers = workloads.layer_keys(seed=14, n_layers=5, N=333, n_h=3, d_h=32)
    want = _oracle(layers)
    got, layer = _run(layers, 0.05, torch.bfloat16, 3, 32)
    assert np.abs(got - want).max() <= _tolerance(96)
    assert layer == orc.select_layer([f64(K) for K in layers], 0.05)


def test_spread_special_cases():
    row = torch.from_numpy(np.random.default_rng(3).standard_normal((1, 512))).to(torch.bfloat16)
    same = (row.float() * torch.tensor([[1.0], [2.0], [0.5], [4.0]])).to(torch.bfloat16)   # exact multiples
    opp = torch.cat([same, -same])
    ortho = torch.zeros((5, 512), dtype=torch.bfloat16)
    ortho[torch.arange(5), torch.arange(5) * 100] = torch.tensor([1.0, 3.0, 0.5, 2.0, 7.0], dtype=torch.bfloat16)
    for K, want in ((same, 0.0), (opp, 2.0), (ortho, 1.0)):
        got, _ = _run([K], 0.5, torch.bfloat16, 4, 128)
        assert abs(got[0] - want) <= 2.0 ** -20 and abs(orc.max_key_distance(f64(K)) - want) < 1e-12


def test_spread_at_full_size_ten_layers():
    layers = workloads.layer_keys(seed=5, n_layers=10, N=7290)
    want = _oracle(layers)
    got, layer = _run(layers, 0.3, torch.bfloat16, 4, 128)
    assert np.abs(got - want).max() <= _tolerance(512)
    assert layer == orc.select_layer([f64(K) for K in layers], 0.3)
    assert layer not in (-1, int(np.argmax(want)))        # earliest qualifying, not the widest


def test_spread_rejects_bad_arguments():
    import ctypes as C
    from paper_2504_08966_b200 import binding as pb
    ctx = pb.Context(64, 4, 4, 128, torch.bfloat16, torch.bfloat16)
    K = torch.zeros((64, 512), dtype=torch.bfloat16, device="cuda")
    md = torch.zeros(4, dtype=torch.float32, device="cuda")
    ctx.ensure_workspace(1, 64)
    w, n = ctx._ws()
    L = pb.lib()
    arr = (C.c_void_p * 1)(K.data_ptr())
    none = (C.c_void_p * 1)(None)
    odd = (C.c_void_p * 1)(K.data_ptr() + 2)
    vp = lambda t: C.c_void_p(t.data_ptr())
    call = lambda a, nl, ld, N, thr, out, ws, nb: L.pact_key_spread(ctx.handle, a, nl, ld, N, thr, out, None, ws, nb, None)
    assert call(arr, 1, 512, 64, 0.5, vp(md), w, n) == 0
    assert call(arr, 0, 512, 64, 0.5, vp(md), w, n) == -1
    assert call(arr, 1, 512, 0, 0.5, vp(md), w, n) == -1
    assert call(arr, 1, 100, 64, 0.5, vp(md), w, n) == -1
    assert call(none, 1, 512, 64, 0.5, vp(md), w, n) == -1
    assert call(odd, 1, 512, 64, 0.5, vp(md), w, n) == -1
    assert call(arr, 1, 512, 64, float("nan"), vp(md), w, n) == -1
    assert call(arr, 1, 512, 64, 0.5, None, w, n) == -1
    assert call(arr, 1, 512, 64, 0.5, vp(md), w, C.c_size_t(1024)) == -3
    torch.cuda.synchronize()
