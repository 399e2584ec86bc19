"""Shared test helpers: widen workload tensors for the oracle and run it on one image."""
import numpy as np
import torch

from oracle import pact_oracle as orc


def f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a bf16/fp32 tensor to float64."""
    return t.to(torch.float64).numpy()


def oracle_image(wl, img, **over):
    """Run the oracle's Algorithm 3 on one image of a workload."""
    kw = dict(lam=wl.lam, d_c=wl.d_c, d_n=wl.d_n, alpha=wl.alpha)
    kw.update(over)
    Kc = img.K_clu if img.K_clu is not None else img.K
    return orc.pact_reduce(f64(img.H), f64(img.K), f64(img.Q), f64(Kc), img.P.numpy(),
                           img.vis_start, img.N, wl.n_qh, wl.n_kvh, **kw)


# ---------------------------------------------------------------------------------------------
# GPU side (imports the binding lazily so that CPU-only collection never loads CUDA)
# ---------------------------------------------------------------------------------------------

def gpu_reduce(wl, out_dtype=None, params=None, **over):
    """Runs pact_reduce on every image of a workload; returns (list of per-image dicts, ctx)."""
    from paper_2504_08966_b200 import binding as pb
    out_dtype = out_dtype or wl.dtype
    ctx = pb.Context(wl.d, wl.n_qh, wl.n_kvh, wl.d_h, wl.dtype, out_dtype)
    ims = [pb.device_image(img, out_dtype) for img in wl.images]
    if params is None:
        kw = dict(lam=wl.lam, d_c=wl.d_c, d_n=wl.d_n, alpha=wl.alpha)
        kw.update(over)
        params = pb.make_params(**kw)
    ctx.pact_reduce(ims, params)
    torch.cuda.synchronize()
    outs = []
    for im in ims:
        cnt = im.counters.cpu().numpy()
        n_out = int(cnt[pb.CNT["n_out"]])
        outs.append({
            "counters": cnt, "n_out": n_out, "q": int(cnt[pb.CNT["q"]]), "C": int(cnt[pb.CNT["C"]]),
            "r": int(cnt[pb.CNT["r"]]), "discarded": int(cnt[pb.CNT["discarded"]]),
            "status": int(cnt[pb.CNT["status"]]), "sweeps": int(cnt[pb.CNT["sweeps"]]),
            "band_dc": int(cnt[pb.CNT["band_dc"]]), "band_adc": int(cnt[pb.CNT["band_adc"]]),
            "label": im.label.cpu().numpy(), "keep": im.keep.cpu().numpy().astype(bool),
            "score": im.score.cpu().numpy(),
            "H_out": im.H_out[:n_out].to(torch.float64).cpu().numpy(),
            "H_out_raw": im.H_out[:n_out].cpu(),
            "P_out": im.P_out[:n_out].cpu().numpy(), "size_out": im.size_out[:n_out].cpu().numpy(),
            "logw_out": im.logw_out[:n_out].cpu().numpy().astype(np.float64),
        })
    return outs, ctx


def bf16_round(x: np.ndarray) -> np.ndarray:
    """float64 -> nearest bf16 (ties to even), returned as float64."""
    return torch.from_numpy(np.ascontiguousarray(x)).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()


def fragile_report(o, wl_d_c=None, alpha=None):
    """The oracle's float64 count of near-threshold decisions of one image (see orc.fragile_decisions)."""
    return o["fragile"]


def compare_image(o, g, img, out_is_bf16, check_scores=True):
    """Element-by-element comparison of the CUDA result g with the oracle result o.
    Returns a list of mismatch descriptions (empty = parity)."""
    bad = []
    if g["status"] != 0:
        bad.append(f"device status {g['status']}")
    if check_scores:
        rel = np.abs(g["score"].astype(np.float64) - o["scores"]) / np.maximum(np.abs(o["scores"]), 1e-300)
        if rel.max() > 2e-7:
            bad.append(f"score rel err {rel.max():.3e}")
    if not np.array_equal(g["keep"], o["keep"]):
        bad.append(f"keep mask differs at {np.nonzero(g['keep'] != o['keep'])[0][:8]}")
        return bad
    for k in ("q", "C", "r", "discarded", "n_out"):
        if g[k] != o[k]:
            bad.append(f"{k}: gpu {g[k]} oracle {o[k]}")
    if not np.array_equal(g["label"], o["label"]):
        idx = np.nonzero(g["label"] != o["label"])[0]
        bad.append(f"labels differ at {idx.size} tokens, first {idx[:8]}")
        return bad
    if g["n_out"] != o["n_out"]:
        return bad
    if not np.array_equal(g["P_out"], o["P_out"]):
        bad.append("P_out differs")
    if not np.array_equal(g["size_out"], o["size_out"]):
        bad.append("size_out differs")
    # Eq. 11 bias: fp32 logarithm of an exact integer, two units in the last place
    if (np.abs(g["logw_out"] - o["logw_out"]) > 2.4e-7 * np.maximum(o["logw_out"], 1.0)).any():
        bad.append("logw_out differs from log(size_out)")
    ref = o["H_out"]
    if out_is_bf16:
        want = bf16_round(ref)
        # within one bf16 ulp of the rounded oracle value
        ulp = np.maximum(np.abs(want), 2.0 ** -126) * 2.0 ** -7
        err = np.abs(g["H_out"] - want)
        if (err > ulp).any():
            bad.append(f"H_out (bf16) off by more than 1 ulp at {int((err > ulp).sum())} elements")
        vs, C = img.vis_start, o["C"]
        text = np.r_[0:vs, vs + C:o["n_out"]]
        if not np.array_equal(g["H_out"][text], ref[text]):
            bad.append("text rows not bit-identical")
    else:
        num = np.abs(g["H_out"] - ref).max(axis=1)
        den = np.maximum(np.abs(ref).max(axis=1), 1e-300)
        if (num / den).max() > 2e-3:
            bad.append(f"H_out rel err {(num / den).max():.3e} > 2e-3")
    return bad
