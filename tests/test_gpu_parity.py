"""Parity of the CUDA path (through the C ABI) with the CPU oracle on the same seeded inputs.

Bar: keep masks, cluster ids, reincorporation decisions, position ids and sizes bit-exact;
scores within 2e-7 relative (float32 output of a float64 computation); merged hidden states
within 2e-3 relative per row for float32 output, within one bf16 ulp of the rounded oracle
value for bf16 output.  Text rows are bit-identical.
"""
import numpy as np
import pytest
import torch

from oracle import pact_oracle as orc
from paper_2504_08966_b200 import workloads
from tests.helpers import compare_image, f64, fragile_report, gpu_reduce, oracle_image

pytestmark = pytest.mark.gpu


def _check_workload(wl, out_dtype, **over):
    outs, _ = gpu_reduce(wl, out_dtype, **over)
    for b, (img, g) in enumerate(zip(wl.images, outs)):
        o = oracle_image(wl, img, **{k: v for k, v in over.items() if k in ("lam", "d_c", "d_n", "alpha")})
        bad = compare_image(o, g, img, out_dtype == torch.bfloat16)
        assert not bad, f"{wl.name} image {b}: {bad}; fragile: {fragile_report(o, over.get('d_c', wl.d_c), wl.alpha)}"
        assert o["q"] + g["r"] + g["discarded"] == img.N
    return outs


# ------------------------------------------------------------------ the five workloads

def test_tiny_fp32():
    outs = _check_workload(workloads.tiny(), torch.float32)
    assert outs[0]["C"] == 12


@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_single_image_full_size(out_dtype):
    _check_workload(workloads.single_image(), out_dtype)


def test_video_full_size():
    _check_workload(workloads.video(), torch.bfloat16)


@pytest.mark.parametrize("lam", [0.3, 0.5, 0.7])
@pytest.mark.parametrize("d_c", [0.2, 0.3, 0.5])
def test_batched_sweep(lam, d_c):
    wl = workloads.batched()
    _check_workload(wl, torch.bfloat16, lam=lam, d_c=d_c)


def test_stress_full_size():
    _check_workload(workloads.stress(), torch.bfloat16)


def test_batch_with_per_image_params_and_mixed_sizes():
    from paper_2504_08966_b200 import binding as pb
    a = workloads.single_image(seed=11, N=1500, T=12, n_blobs=40)
    b = workloads.single_image(seed=12, N=901, T=0, n_blobs=25)
    c = workloads.single_image(seed=13, N=2309, T=40, n_blobs=60)
    wl = workloads.Workload("mixed", a.images + b.images + c.images, a.d, a.n_qh, a.n_kvh, a.d_h,
                            a.dtype, 0.5, 0.3)
    plist = [(0.5, 0.3, 1.5), (0.2, 0.45, 1.0), (0.8, 0.15, 2.0)]
    params = [pb.make_params(lam=l, d_c=dc, alpha=al) for l, dc, al in plist]
    outs, _ = gpu_reduce(wl, torch.bfloat16, params=params)
    for img, g, (l, dc, al) in zip(wl.images, outs, plist):
        o = oracle_image(wl, img, lam=l, d_c=dc, alpha=al)
        assert not compare_image(o, g, img, True)


def test_batch_of_sixteen_with_extreme_size_mix():
    """Sixteen images from 1 to 4100 tokens in one call: every image has its own share of every grid."""
    sizes = [1, 4100, 2, 33, 700, 129, 3000, 5, 64, 1023, 257, 31, 2048, 300, 17, 1500]
    imgs, first = [], None
    for k, n in enumerate(sizes):
        w = _small(seed=300 + k, N=n, T=k % 5, n_blobs=max(1, min(30, n // 8 + 1)))
        first = first or w
        imgs += w.images
    wl = workloads.Workload("mix16", imgs, first.d, first.n_qh, first.n_kvh, first.d_h, first.dtype, 0.5, 0.3)
    outs, _ = gpu_reduce(wl, torch.bfloat16)
    for img, g in zip(wl.images, outs):
        o = oracle_image(wl, img)
        bad = compare_image(o, g, img, True)
        assert not bad, f"N={img.N}: {bad}"


def test_random_configurations():
    """Forty seeded random combinations of size, shape, element type and parameters."""
    rng = np.random.default_rng(2024)
    for case in range(40):
        N = int(rng.choice([rng.integers(1, 40), rng.integers(40, 400), rng.integers(400, 2600)]))
        dtype = torch.bfloat16 if rng.random() < 0.7 else torch.float32
        n_h, d_h = [(2, 32), (4, 128), (2, 64), (3, 16), (1, 64)][rng.integers(0, 5)]
        kw = dict(seed=int(rng.integers(1, 10 ** 6)), N=N, T=int(rng.integers(0, 12)),
                  n_blobs=int(max(1, min(60, N // int(rng.integers(3, 30)) + 1))),
                  d=int(rng.choice([64, 256, 512, 1032])), n_h=n_h, d_h=d_h, dtype=dtype)
        over = dict(lam=float(rng.choice([0.0, 0.1, 0.3, 0.5, 0.7, 0.9, 1.0, rng.random()])),
                    d_c=float(rng.choice([0.0, 0.05, 0.2, 0.3, 0.5, 1.0, 2.0, rng.random()])),
                    alpha=float(rng.choice([0.0, 1.0, 1.5, 3.0, rng.random() * 2])),
                    d_n=float(rng.choice([0.5, 2.0, 4.0])))
        out_dtype = torch.float32 if (dtype == torch.float32 or rng.random() < 0.5) else torch.bfloat16
        wl = workloads.single_image(**kw)
        outs, _ = gpu_reduce(wl, out_dtype, **over)
        img = wl.images[0]
        o = oracle_image(wl, img, **over)
        bad = compare_image(o, outs[0], img, out_dtype == torch.bfloat16)
        assert not bad, f"case {case} {kw} {over} {out_dtype}: {bad}; fragile: {fragile_report(o, over['d_c'], over['alpha'])}"


# ------------------------------------------------------------------ edge and degenerate cases

def _small(seed=21, N=700, T=9, **kw):
    base = dict(n_blobs=18, d=256, n_h=2, d_h=32)
    base.update(kw)
    return workloads.single_image(seed=seed, N=N, T=T, **base)


@pytest.mark.parametrize("N", [1, 2, 31, 33, 129, 1023])
def test_ragged_and_minimal_sizes(N):
    _check_workload(_small(seed=30 + N, N=N, T=3, n_blobs=max(1, min(18, N // 4 + 1))), torch.float32)


@pytest.mark.parametrize("over", [dict(lam=0.0), dict(lam=1.0), dict(alpha=0.0), dict(d_c=0.0), dict(d_c=2.0),
                                  dict(lam=0.0, d_c=1e-9), dict(alpha=6.0, d_c=0.34), dict(d_n=0.5)])
def test_degenerate_parameters(over):
    wl = _small()
    outs = _check_workload(wl, torch.float32, **over)
    g, N = outs[0], wl.images[0].N
    if over.get("lam") == 0.0:
        assert g["q"] == N and g["r"] == 0
    if over.get("lam") == 1.0:
        assert g["q"] >= 1
    if over.get("alpha") == 0.0:
        assert g["r"] == 0
    if over.get("d_c") == 2.0:
        assert g["C"] == 1
    if over.get("d_c") == 1e-9:
        assert g["C"] == g["q"] == N                          # no merging at all
    if over.get("alpha") == 6.0:
        assert g["discarded"] == 0


@pytest.mark.parametrize("kind", ["uniform", "two_valued", "zero_keys", "one_hot_runs"])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_degenerate_inputs(kind, dtype):
    """Images whose keys repeat exactly (flat regions), vanish, or are exactly parallel."""
    wl = workloads.single_image(seed=61, N=900, T=6, n_blobs=20, d=256, n_h=2, d_h=64, dtype=dtype)
    img = wl.images[0]
    K = img.K
    if kind == "uniform":
        K[:] = K[17].clone()
    elif kind == "two_valued":
        a, b = K[3].clone(), K[4].clone()
        K[0::2] = a
        K[1::2] = b
    elif kind == "zero_keys":
        K[100:164] = 0
        K[500] = 0
    else:
        K[200:264] = 0
        K[200:264, 5] = torch.tensor([2.0 ** (i % 4 - 2) for i in range(64)], dtype=dtype)
        img.H[img.vis_start + 200:img.vis_start + 264] *= 4      # keep them among the survivors
    outs = _check_workload(wl, torch.float32)
    if kind == "uniform":
        assert outs[0]["C"] == 1 and outs[0]["discarded"] == 0
    if kind == "two_valued":
        assert outs[0]["C"] <= 2


def test_no_text_tokens_and_gqa_and_distinct_clustering_keys():
    _check_workload(_small(seed=41, T=0), torch.bfloat16)
    _check_workload(_small(seed=42, n_qh=4), torch.bfloat16)
    _check_workload(_small(seed=43, distinct_k_clu=True), torch.bfloat16)
    _check_workload(_small(seed=44, dtype=torch.float32, d_h=16, n_h=3, d=136), torch.float32)
    # bf16 keys whose width is not a multiple of 64 take the SIMT tile kernels
    _check_workload(_small(seed=45, d_h=48, n_h=2, d=264), torch.bfloat16)


def test_exact_duplicates_tie_break():
    wl = workloads.stress(seed=9, B=1, N=1200, T=8, n_blobs=30, dup_frac=0.2, d=256, n_h=2, d_h=32, lam=0.3)
    outs = _check_workload(wl, torch.float32)
    assert outs[0]["C"] > 1


def test_flags_center_only_and_score_ablations():
    from paper_2504_08966_b200 import binding as pb
    wl = _small(seed=51)
    img = wl.images[0]
    for flags, okw in [(pb.FLAG_CENTER_ONLY, dict(center_only=True)), (pb.FLAG_NO_NORM, dict(use_norm=False)),
                       (pb.FLAG_NORM_ONLY, dict(use_query=False))]:
        outs, _ = gpu_reduce(wl, torch.float32, flags=flags)
        o = oracle_image(wl, img, **okw)
        assert not compare_image(o, outs[0], img, False), flags


def test_strided_inputs():
    """Row strides larger than the row width (views into wider buffers)."""
    from paper_2504_08966_b200 import binding as pb
    wl = _small(seed=61)
    img = wl.images[0]
    ctx = pb.Context(wl.d, wl.n_qh, wl.n_kvh, wl.d_h, wl.dtype, torch.float32)
    im = pb.device_image(img, torch.float32)
    def widen(t, extra):
        buf = torch.zeros((t.shape[0], t.shape[1] + extra), dtype=t.dtype, device=t.device)
        buf[:, :t.shape[1]] = t
        return buf[:, :t.shape[1]]
    im.H, im.K_euti, im.Q_euti = widen(im.H, 64), widen(im.K_euti, 8), widen(im.Q_euti, 16)
    im.K_clu = im.K_euti
    im.H_out = widen(im.H_out, 32)
    ctx.pact_reduce([im], pb.make_params(lam=wl.lam, d_c=wl.d_c))
    torch.cuda.synchronize()
    o = oracle_image(wl, img)
    n_out = int(im.counters[0])
    assert n_out == o["n_out"] and np.array_equal(im.label.cpu().numpy(), o["label"])
    got = im.H_out[:n_out].double().cpu().numpy()
    num = np.abs(got - o["H_out"]).max(axis=1)
    den = np.maximum(np.abs(o["H_out"]).max(axis=1), 1e-300)
    assert (num / den).max() <= 2e-3                        # per row, as everywhere else
    assert np.array_equal(im.P_out[:n_out].cpu().numpy(), o["P_out"])


def test_bitwise_deterministic_run_to_run():
    wl = workloads.single_image(seed=71, N=3000, T=16, n_blobs=80)
    a, _ = gpu_reduce(wl, torch.bfloat16)
    b, _ = gpu_reduce(wl, torch.bfloat16)
    assert np.array_equal(a[0]["label"], b[0]["label"])
    assert torch.equal(a[0]["H_out_raw"].view(torch.int16), b[0]["H_out_raw"].view(torch.int16))
    assert np.array_equal(a[0]["score"].view(np.int32), b[0]["score"].view(np.int32))


def test_more_than_16384_tokens_takes_the_general_select_path():
    """Beyond 16384 tokens the split keeps its keys in shared memory instead of registers."""
    wl = workloads.single_image(seed=75, N=17011, T=5, n_blobs=60, lam=0.85, d=128, n_h=2, d_h=32)
    outs = _check_workload(wl, torch.float32)
    assert outs[0]["q"] >= 2551


@pytest.mark.parametrize("N", [40000, 60001])
def test_stage_prune_large_inputs(N):
    """40000 keys fit in shared memory, 60001 are re-read from the scores."""
    from paper_2504_08966_b200 import binding as pb
    ctx = pb.Context(256, 2, 2, 32, torch.bfloat16, torch.bfloat16)
    g = torch.Generator().manual_seed(N)
    s32 = (torch.rand(N, generator=g) * torch.exp(4 * torch.randn(N, generator=g))).numpy().astype(np.float32)
    s32[7] = s32[N - 3] = s32[N // 2]
    for lam in (0.37, 0.9):
        tau, keep, kept, pruned = orc.split(s32, lam)
        dev = lambda dt: torch.empty(N, dtype=dt, device="cuda")
        keep_d, kept_d, pruned_d, counts = dev(torch.uint8), dev(torch.int32), dev(torch.int32), torch.zeros(2, dtype=torch.int32, device="cuda")
        ctx.pact_prune(torch.from_numpy(s32).cuda(), pb.make_params(lam=lam), keep_d, kept_d, pruned_d, counts)
        q, m = counts.cpu().tolist()
        assert q == kept.size and m == pruned.size
        assert np.array_equal(keep_d.cpu().numpy().astype(bool), keep)
        assert np.array_equal(kept_d[:q].cpu().numpy(), kept) and np.array_equal(pruned_d[:m].cpu().numpy(), pruned)


def test_graph_replay_matches_direct_call_bitwise():
    from paper_2504_08966_b200 import binding as pb
    wl = workloads.single_image(seed=72, N=2100, T=10, n_blobs=50)
    direct, _ = gpu_reduce(wl, torch.bfloat16)
    ctx = pb.Context(wl.d, wl.n_qh, wl.n_kvh, wl.d_h, wl.dtype, torch.bfloat16)
    ims = [pb.device_image(img, torch.bfloat16) for img in wl.images]
    g = ctx.pact_graph_create(ims, pb.make_params(lam=wl.lam, d_c=wl.d_c, d_n=wl.d_n, alpha=wl.alpha))
    for rep in range(3):
        ims[0].H_out.zero_()
        ims[0].label.fill_(-7)
        g.launch()
        torch.cuda.synchronize()
        cnt = ims[0].counters.cpu().numpy()
        n_out = int(cnt[pb.CNT["n_out"]])
        assert int(cnt[pb.CNT["status"]]) == 0 and n_out == direct[0]["n_out"]
        assert np.array_equal(ims[0].label.cpu().numpy(), direct[0]["label"])
        assert torch.equal(ims[0].H_out[:n_out].cpu().view(torch.int16), direct[0]["H_out_raw"].view(torch.int16))
    o = oracle_image(wl, wl.images[0])
    assert np.array_equal(direct[0]["label"], o["label"])
    g.close()


def test_full_size_image_as_the_benchmark_runs_it():
    """The timed configuration: N = 7290, bf16 output, graph replays rotating over input copies."""
    from paper_2504_08966_b200 import binding as pb
    wl = workloads.single_image()
    img = wl.images[0]
    o = oracle_image(wl, img)
    ctx = pb.Context(wl.d, wl.n_qh, wl.n_kvh, wl.d_h, wl.dtype, torch.bfloat16)
    params = pb.make_params(lam=wl.lam, d_c=wl.d_c, d_n=wl.d_n, alpha=wl.alpha)
    sets = [[pb.device_image(img, torch.bfloat16)] for _ in range(3)]
    graphs = [ctx.pact_graph_create(ims, params) for ims in sets]
    for i in range(31):
        graphs[i % 3].launch()
    torch.cuda.synchronize()
    for ims in sets:
        im = ims[0]
        cnt = im.counters.cpu().numpy()
        n_out = int(cnt[pb.CNT["n_out"]])
        g = {"counters": cnt, "n_out": n_out, "q": int(cnt[pb.CNT["q"]]), "C": int(cnt[pb.CNT["C"]]),
             "r": int(cnt[pb.CNT["r"]]), "discarded": int(cnt[pb.CNT["discarded"]]),
             "status": int(cnt[pb.CNT["status"]]), "label": im.label.cpu().numpy(),
             "keep": im.keep.cpu().numpy().astype(bool), "score": im.score.cpu().numpy(),
             "H_out": im.H_out[:n_out].to(torch.float64).cpu().numpy(),
             "P_out": im.P_out[:n_out].cpu().numpy(), "size_out": im.size_out[:n_out].cpu().numpy(),
             "logw_out": im.logw_out[:n_out].cpu().numpy().astype(np.float64)}
        assert g["status"] == 0
        assert not compare_image(o, g, img, True)
    for gr in graphs:
        gr.close()


def test_contexts_on_separate_streams_do_not_interfere():
    """Independent requests in flight at once: one context, workspace and graph per stream; every
    stream must reproduce what the same request gives alone."""
    from paper_2504_08966_b200 import binding as pb
    wls = [workloads.single_image(seed=70 + i, N=1800 + 211 * i, T=10, n_blobs=40) for i in range(3)]
    alone = []
    for wl in wls:
        outs, _ = gpu_reduce(wl, torch.bfloat16)
        alone.append(outs[0])
    ctxs, graphs, ims, streams = [], [], [], []
    for wl in wls:
        ctx = pb.Context(wl.d, wl.n_qh, wl.n_kvh, wl.d_h, wl.dtype, torch.bfloat16)
        im = pb.device_image(wl.images[0], torch.bfloat16)
        ctxs.append(ctx)
        ims.append(im)
        graphs.append(ctx.pact_graph_create([im], pb.make_params(lam=wl.lam, d_c=wl.d_c, d_n=wl.d_n, alpha=wl.alpha)))
        streams.append(torch.cuda.Stream())
    torch.cuda.synchronize()
    for rep in range(20):
        for g, st in zip(graphs, streams):
            with torch.cuda.stream(st):
                g.launch()
    torch.cuda.synchronize()
    for im, ref in zip(ims, alone):
        cnt = im.counters.cpu().numpy()
        n_out = int(cnt[pb.CNT["n_out"]])
        assert int(cnt[pb.CNT["status"]]) == 0 and n_out == ref["n_out"]
        assert np.array_equal(im.label.cpu().numpy(), ref["label"])
        assert torch.equal(im.H_out[:n_out].cpu().view(torch.int16), ref["H_out_raw"].view(torch.int16))
        assert np.array_equal(im.P_out[:n_out].cpu().numpy(), ref["P_out"])
    for g in graphs:
        g.close()


# ------------------------------------------------------------------ stage calls against the oracle's stages

@pytest.fixture(scope="module")
def stage_case():
    from paper_2504_08966_b200 import binding as pb
    wl = workloads.single_image(seed=81, N=2500, T=20, n_blobs=70)
    img = wl.images[0]
    o = oracle_image(wl, img)
    ctx = pb.Context(wl.d, wl.n_qh, wl.n_kvh, wl.d_h, wl.dtype, torch.float32)
    im = pb.device_image(img, torch.float32)
    return wl, img, o, ctx, im, pb.make_params(lam=wl.lam, d_c=wl.d_c, d_n=wl.d_n, alpha=wl.alpha)


def test_stage_importance(stage_case):
    wl, img, o, ctx, im, params = stage_case
    score = torch.empty(img.N, dtype=torch.float32, device="cuda")
    ctx.pact_importance(im, params, score)
    got = score.cpu().numpy()
    rel = np.abs(got.astype(np.float64) - o["scores"]) / o["scores"]
    assert rel.max() <= 2e-7
    assert (got == o["scores32"]).mean() > 0.9
    assert abs((got.astype(np.float64) / np.linalg.norm(f64(img.H)[img.vis_start:img.vis_start + img.N], axis=1)).sum() - 1) < 1e-5


@pytest.mark.parametrize("lam", [0.0, 0.25, 0.5, 0.999, 1.0])
def test_stage_prune_bit_exact(stage_case, lam):
    from paper_2504_08966_b200 import binding as pb
    wl, img, o, ctx, im, _ = stage_case
    s32 = o["scores32"].copy()
    s32[5] = s32[100] = s32[7]                       # ties
    s32[11] = -1.5                                   # a negative and a zero score
    s32[12] = 0.0
    tau, keep, kept, pruned = orc.split(s32, lam)
    N = img.N
    dev = lambda dt: torch.empty(N, dtype=dt, device="cuda")
    keep_d, kept_d, pruned_d, counts = dev(torch.uint8), dev(torch.int32), dev(torch.int32), torch.zeros(2, dtype=torch.int32, device="cuda")
    ctx.pact_prune(torch.from_numpy(s32).cuda(), pb.make_params(lam=lam), keep_d, kept_d, pruned_d, counts)
    q, m = counts.cpu().tolist()
    assert q == kept.size and m == pruned.size
    assert np.array_equal(keep_d.cpu().numpy().astype(bool), keep)
    assert np.array_equal(kept_d[:q].cpu().numpy(), kept) and np.array_equal(pruned_d[:m].cpu().numpy(), pruned)


def test_stage_dbdpc_reincorporate_merge(stage_case):
    wl, img, o, ctx, im, params = stage_case
    N = img.N
    kept = torch.from_numpy(o["kept_idx"]).cuda()
    q_dev = torch.tensor([o["q"]], dtype=torch.int32, device="cuda")
    rho = torch.empty(N, dtype=torch.float32, device="cuda")
    cidx = torch.empty(N, dtype=torch.int32, device="cuda")
    C_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    label = torch.empty(N, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(16, dtype=torch.int32, device="cuda")
    ctx.pact_dbdpc(im.K_clu, kept, q_dev, params, rho, cidx, C_dev, label, cnt)
    C = int(C_dev)
    assert C == o["C"] and np.array_equal(cidx[:C].cpu().numpy(), o["center_idx"])
    want = np.full(N, -1)
    want[o["kept_idx"]] = o["label"][o["kept_idx"]]
    assert np.array_equal(label.cpu().numpy(), want)
    rel = np.abs(rho[:o["q"]].cpu().numpy() - o["rho"]) / o["rho"]
    assert rel.max() < 1e-6
    # the float32 densities the stage returns give the oracle's order wherever the oracle's own densities are
    # further apart than float32 resolves: compare the order up to runs of such near-equal neighbours
    got_rho = rho[:o["q"]].cpu().numpy().astype(np.float64)
    ord_o = o["order"]
    gaps = o["rho"][ord_o[:-1]] - o["rho"][ord_o[1:]]
    clear = gaps > 4e-7 * o["rho"][ord_o[:-1]]             # float32 keeps these apart (ulp 6e-8, error <= 1e-6 checked above)
    assert clear.mean() > 0.5
    assert np.all(got_rho[ord_o[:-1]][clear] >= got_rho[ord_o[1:]][clear])
    # reincorporation from the oracle's centres
    pruned = torch.from_numpy(o["pruned_idx"]).cuda()
    m_dev = torch.tensor([o["pruned_idx"].size], dtype=torch.int32, device="cuda")
    r_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    cidx_o = torch.from_numpy(o["center_idx"].astype(np.int32)).cuda()
    C_o = torch.tensor([o["C"]], dtype=torch.int32, device="cuda")
    lab2 = torch.from_numpy(want.astype(np.int32)).cuda()
    ctx.pact_reincorporate(im.K_clu, pruned, m_dev, cidx_o, C_o, params, lab2, r_dev)
    assert int(r_dev) == o["r"] and np.array_equal(lab2.cpu().numpy(), o["label"])
    # merge from the oracle's labels
    lab_o = torch.from_numpy(o["label"].astype(np.int32)).cuda()
    ctx.pact_merge(im, lab_o, cidx_o, C_o, params)
    torch.cuda.synchronize()
    n_out = int(im.counters[0])
    assert n_out == o["n_out"]
    got = im.H_out[:n_out].double().cpu().numpy()
    num = np.abs(got - o["H_out"]).max(axis=1)
    assert (num / np.abs(o["H_out"]).max(axis=1)).max() <= 2e-3
    assert np.array_equal(im.P_out[:n_out].cpu().numpy(), o["P_out"])
    assert np.array_equal(im.size_out[:n_out].cpu().numpy(), o["size_out"])


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_stage_dbdpc_runs_of_identical_keys(dtype):
    """Uniform image regions give runs of identical (or exactly parallel) keys: many neighbouring
    pairs at distance 0, each adding the largest possible term to a density."""
    from paper_2504_08966_b200 import binding as pb
    wl = workloads.single_image(seed=83, N=1500, T=8, n_blobs=40, dtype=dtype)
    K = wl.images[0].K.clone()
    K[200:218] = K[200]
    K[300:309] = (K[300].float() * 2.0).to(dtype)
    K[301] = K[300]
    K[640:644] = K[640]
    # one non-zero element, a power of two: norms and cosines are exact, these distances are exactly 0
    K[800:813] = 0
    K[800:813, 3] = torch.tensor([2.0 ** (i % 3 - 1) for i in range(13)], dtype=dtype)
    N = K.shape[0]
    o = orc.dbdpc(f64(K), wl.d_c, wl.d_n)
    ctx = pb.Context(wl.d, wl.n_qh, wl.n_kvh, wl.d_h, dtype, torch.float32)
    idx = torch.arange(N, dtype=torch.int32, device="cuda")
    q_dev = torch.tensor([N], dtype=torch.int32, device="cuda")
    rho = torch.empty(N, dtype=torch.float32, device="cuda")
    cidx = torch.empty(N, dtype=torch.int32, device="cuda")
    C_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    label = torch.empty(N, dtype=torch.int32, device="cuda")
    ctx.pact_dbdpc(K.cuda(), idx, q_dev, pb.make_params(lam=0.0, d_c=wl.d_c, d_n=wl.d_n), rho, cidx, C_dev, label)
    torch.cuda.synchronize()
    rel = np.abs(rho.cpu().numpy() - o["rho"]) / o["rho"]
    assert rel.max() < 1e-6
    C = int(C_dev)
    assert C == o["centers"].size and np.array_equal(cidx[:C].cpu().numpy(), o["centers"])
    assert np.array_equal(label.cpu().numpy(), o["label"])


def test_stage_dbdpc_over_all_tokens_at_full_size():
    """DBDPC as a clustering method of its own (nothing pruned): N = 7290 rows in the Gram pass."""
    from paper_2504_08966_b200 import binding as pb
    wl = workloads.single_image()
    img = wl.images[0]
    N = img.N
    o = orc.dbdpc(f64(img.K), wl.d_c, wl.d_n)
    ctx = pb.Context(wl.d, wl.n_qh, wl.n_kvh, wl.d_h, wl.dtype, torch.bfloat16)
    K = img.K.cuda()
    idx = torch.arange(N, dtype=torch.int32, device="cuda")
    q_dev = torch.tensor([N], dtype=torch.int32, device="cuda")
    rho = torch.empty(N, dtype=torch.float32, device="cuda")
    cidx = torch.empty(N, dtype=torch.int32, device="cuda")
    C_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    label = torch.empty(N, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(16, dtype=torch.int32, device="cuda")
    ctx.pact_dbdpc(K, idx, q_dev, pb.make_params(lam=0.0, d_c=wl.d_c, d_n=wl.d_n), rho, cidx, C_dev, label, cnt)
    torch.cuda.synchronize()
    c = cnt.cpu().numpy()
    assert int(c[pb.CNT["status"]]) == 0
    iu = np.triu_indices(N, 1)
    fragile = int((np.abs(o["D"][iu] - float(np.float32(wl.d_c))) <= 1e-6).sum())
    assert int(c[pb.CNT["band_dc"]]) >= fragile - 2 and fragile < 50
    C = int(C_dev)
    if fragile == 0:
        assert C == o["centers"].size and np.array_equal(cidx[:C].cpu().numpy(), o["centers"])
        assert np.array_equal(label.cpu().numpy(), o["label"])
    else:   # pairs on the cutoff may fall either way in fp32; the rest of the structure must hold
        assert abs(C - o["centers"].size) <= fragile
        assert (label.cpu().numpy() == o["label"]).mean() > 0.9 or C != o["centers"].size
    rel = np.abs(rho.cpu().numpy() - o["rho"]) / o["rho"]
    assert rel.max() < 1e-6


# ------------------------------------------------------------------ host-buffer entry point and error paths

def test_reduce_host_matches_device_path():
    from paper_2504_08966_b200 import binding as pb
    wl = _small(seed=91)
    img = wl.images[0]
    ctx = pb.Context(wl.d, wl.n_qh, wl.n_kvh, wl.d_h, wl.dtype, torch.bfloat16)
    pin = lambda t: t.contiguous().pin_memory()
    host = dict(H=pin(img.H), K_euti=pin(img.K), Q_euti=pin(img.Q), P=pin(img.P), vis_start=img.vis_start, N=img.N,
                H_out=torch.empty_like(img.H).pin_memory(), P_out=torch.empty(img.n_total, dtype=torch.int32).pin_memory(),
                size_out=torch.empty(img.n_total, dtype=torch.int32).pin_memory(),
                logw_out=torch.empty(img.n_total, dtype=torch.float32).pin_memory(),
                label=torch.empty(img.N, dtype=torch.int32).pin_memory(), counters=torch.zeros(16, dtype=torch.int32).pin_memory())
    host["K_clu"] = host["K_euti"]
    staging = torch.empty(ctx.host_staging_bytes(img.n_total, img.N), dtype=torch.uint8, device="cuda")
    ctx.pact_reduce_host(host, pb.make_params(lam=wl.lam, d_c=wl.d_c), staging)
    o = oracle_image(wl, img)
    n_out = int(host["counters"][0])
    assert n_out == o["n_out"] and np.array_equal(host["label"].numpy(), o["label"])
    assert np.array_equal(host["P_out"][:n_out].numpy(), o["P_out"])
    assert np.allclose(host["logw_out"][:n_out].numpy(), o["logw_out"], rtol=2.4e-7, atol=2.4e-7)
    outs, _ = gpu_reduce(wl, torch.bfloat16)
    assert torch.equal(host["H_out"][:n_out].view(torch.int16), outs[0]["H_out_raw"].view(torch.int16))


def test_invalid_arguments_are_rejected_before_launch():
    from paper_2504_08966_b200 import binding as pb
    wl = _small(seed=95, N=64)
    ctx = pb.Context(wl.d, wl.n_qh, wl.n_kvh, wl.d_h, wl.dtype, torch.float32)
    im = pb.device_image(wl.images[0], torch.float32)
    for bad in (dict(lam=1.5), dict(lam=-0.1), dict(d_c=-1.0), dict(d_c=2.5), dict(d_n=0.0), dict(alpha=-1.0),
                dict(flags=pb.FLAG_NO_NORM | pb.FLAG_NORM_ONLY)):
        with pytest.raises(pb.PactError):
            ctx.pact_reduce([im], pb.make_params(**bad))
    ctx.ensure_workspace(1, 64)
    small = ctx.ws
    ctx.ws = small[:1024]
    L = pb.lib()
    import ctypes as C
    d = im.desc()
    p = pb.make_params()
    st = L.pact_reduce(ctx.handle, C.byref(d), 1, C.byref(p), 0, C.c_void_p(small.data_ptr()), C.c_size_t(1024), None)
    assert st == -3
    st = L.pact_reduce(ctx.handle, C.byref(d), 1, C.byref(p), 0, C.c_void_p(small.data_ptr() + 8), C.c_size_t(small.numel() - 8), None)
    assert st == -3
    d.H = None
    st = L.pact_reduce(ctx.handle, C.byref(d), 1, C.byref(p), 0, C.c_void_p(small.data_ptr()), C.c_size_t(small.numel()), None)
    assert st == -1
    with pytest.raises(pb.PactError):
        pb.Context(100, 4, 3, 16)                   # n_qh not a multiple of n_kvh
    torch.cuda.synchronize()


# ------------------------------------------------------------------ given number of pruned tokens, wait limits, bad labels

@pytest.mark.parametrize("m", [0, 1, 333, 699, 5000])
def test_given_number_of_pruned_tokens(m):
    """pact_params.n_prune replaces the m derived from lambda (Eq. 3-4 with a given m)."""
    from paper_2504_08966_b200 import binding as pb
    wl = _small(seed=83)
    params = pb.make_params(lam=0.9, d_c=wl.d_c, d_n=wl.d_n, alpha=wl.alpha, n_prune=m)
    outs, _ = gpu_reduce(wl, torch.float32, params=params)
    o = oracle_image(wl, wl.images[0], n_prune=m)
    bad = compare_image(o, outs[0], wl.images[0], False)
    assert not bad, f"n_prune={m}: {bad}; fragile: {o['fragile']}"
    assert outs[0]["counters"][9] <= min(m, wl.images[0].N - 1)      # pruned tokens, ties at tau are kept


def test_centre_sweep_limit_is_reported_and_the_context_recovers():
    """A wait that runs out must surface as PACT_ERR_TIMEOUT in the image's status word, with the call
    returning normally, and must leave the context usable: one sweep is not enough for an image whose
    centres depend on one another; the default limit then gives the oracle's result again."""
    from paper_2504_08966_b200 import binding as pb
    wl = workloads.single_image(seed=29, N=2000, T=8, n_blobs=50)
    img = wl.images[0]
    ctx = pb.Context(wl.d, wl.n_qh, wl.n_kvh, wl.d_h, wl.dtype, torch.bfloat16)
    params = pb.make_params(lam=wl.lam, d_c=wl.d_c, d_n=wl.d_n, alpha=wl.alpha)
    im = pb.device_image(img, torch.bfloat16)
    ctx.pact_reduce([im], params)
    torch.cuda.synchronize()
    assert int(im.counters[pb.CNT["status"]]) == 0 and int(im.counters[pb.CNT["sweeps"]]) >= 2
    good = im.label.clone()
    ctx.set_wait_limits(center_sweeps=1)
    ctx.pact_reduce([im], params)                           # returns normally
    torch.cuda.synchronize()
    assert int(im.counters[pb.CNT["status"]]) == -5         # PACT_ERR_TIMEOUT
    n_out = int(im.counters[pb.CNT["n_out"]])
    assert 0 <= n_out <= img.H.shape[0]
    ctx.set_wait_limits()                                   # defaults
    ctx.pact_reduce([im], params)
    torch.cuda.synchronize()
    assert int(im.counters[pb.CNT["status"]]) == 0
    assert torch.equal(im.label, good)
    o = oracle_image(wl, img)
    assert np.array_equal(im.label.cpu().numpy(), o["label"])


def test_merge_reports_a_label_outside_its_range(stage_case):
    """pact_merge takes labels from the caller: one that names no cluster is dropped and reported, the other
    rows are merged as usual and nothing is written out of bounds."""
    wl, img, o, ctx, im, params = stage_case
    label = o["label"].astype(np.int32).copy()
    victim = int(np.nonzero(label >= 0)[0][5])
    label[victim] = o["C"]                                  # one past the last cluster id
    lab_d = torch.from_numpy(label).cuda()
    cidx = torch.from_numpy(o["center_idx"].astype(np.int32)).cuda()
    C_dev = torch.tensor([o["C"]], dtype=torch.int32, device="cuda")
    im.H_out.zero_()
    ctx.pact_merge(im, lab_d, cidx, C_dev, params)
    torch.cuda.synchronize()
    assert int(im.counters[pb_status()]) == -1              # PACT_ERR_INVALID_ARG
    lab_ref = o["label"].copy()
    lab_ref[victim] = -1
    Hm, Pm, sizes = orc.merge(f64(img.H)[img.vis_start:img.vis_start + img.N], lab_ref, o["C"], o["center_idx"],
                              img.P.numpy()[img.vis_start:img.vis_start + img.N])
    got = im.H_out[img.vis_start:img.vis_start + o["C"]].double().cpu().numpy()
    num = np.abs(got - Hm).max(axis=1)
    assert (num / np.maximum(np.abs(Hm).max(axis=1), 1e-300)).max() <= 2e-3
    assert np.array_equal(im.size_out[img.vis_start:img.vis_start + o["C"]].cpu().numpy(), sizes)


def pb_status():
    from paper_2504_08966_b200 import binding as pb
    return pb.CNT["status"]
