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
