"""Seeded synthetic inputs for the PACT reduction step.

This module only draws random numbers and lays them out as the tensors the
method reads (hidden states H, keys K, queries Q, position ids P).  It holds
none of the method's arithmetic (no scores, distances, densities, clusters):
the CPU oracle and the CUDA path both receive what is generated here and
share nothing else.

The paper evaluates on activations of LLaVA-OneVision-7B at layer L=4
(hidden 3584, 4 KV heads x 128).  Neither the weights nor the datasets are
available offline, so these generators stand in for them and reproduce
shapes and coarse statistics only: many visual tokens per image, strongly
redundant keys (blobs and near-duplicates), and a wide spread of
hidden-state norms.

Construction shared by all workloads
------------------------------------
* latent ``z_i`` in R^{d_k}: a unit-norm blob centre plus isotropic noise of
  expected radius ``sigma`` (per-coordinate std ``sigma / sqrt(d_k)``), so the
  cosine between two members of one blob is about ``1 / (1 + sigma^2)``;
* keys ``K_i = g_i * z_i`` with a positive gain ``g_i ~ LogNormal(0, 0.25)``
  (irrelevant to a cosine, relevant to the logits);
* queries ``Q_i = z_i R_q + 0.1 * noise`` with a seeded Gaussian ``R_q``;
* hidden states ``H_i = norm_i * normalise(z_i R_h)`` with a seeded Gaussian
  ``R_h`` and a per-token norm drawn from the workload's norm law;
* position ids ``0 .. n_total-1``; text rows are random and sit before and
  after the visual span: ``[T // 4 text][N visual][T - T // 4 text]``.

Everything is drawn in float64 with ``numpy.random.default_rng(seed)`` and
then rounded once to the workload dtype (bf16 or fp32).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List

import numpy as np
import torch


@dataclass
class Image:
    """One independent unit (an image or a video clip)."""

    H: torch.Tensor        # [n_total, d]
    K: torch.Tensor        # [N, d_k]   keys (used both pre- and post-RoPE: no RoPE is modelled)
    Q: torch.Tensor        # [N, n_qh * d_h]
    P: torch.Tensor        # [n_total] int32
    n_total: int
    vis_start: int
    N: int
    K_clu: torch.Tensor | None = None   # optional distinct post-RoPE keys


@dataclass
class Workload:
    name: str
    images: List[Image]
    d: int
    n_qh: int
    n_kvh: int
    d_h: int
    dtype: torch.dtype
    lam: float
    d_c: float
    d_n: float = 2.0
    alpha: float = 1.5
    note: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def d_k(self) -> int:
        return self.n_kvh * self.d_h


# --------------------------------------------------------------------------
# building blocks (random draws only)
# --------------------------------------------------------------------------

def _unit_rows(x: np.ndarray) -> np.ndarray:
    return x / np.linalg.norm(x, axis=1, keepdims=True)


def _blob_latents(rng, n, centres, sigmas, which=None):
    """n latents around the given unit centres; sigmas is per-centre radius."""
    d_k = centres.shape[1]
    if which is None:
        which = rng.integers(0, centres.shape[0], size=n)
    noise = rng.standard_normal((n, d_k)) * (np.asarray(sigmas)[which, None] / np.sqrt(d_k))
    return centres[which] + noise, which


def _assemble(rng, z, norms, d, n_q_cols, T, dtype, proj_seed):
    """Turn latents and norms into one Image (K, Q, H, P, text rows)."""
    N, d_k = z.shape
    prng = np.random.default_rng(proj_seed)
    R_q = prng.standard_normal((d_k, n_q_cols)) / np.sqrt(d_k)
    R_h = prng.standard_normal((d_k, d)) / np.sqrt(d_k)
    gain = rng.lognormal(0.0, 0.25, size=N)
    K = z * gain[:, None]
    Q = z @ R_q + 0.1 * rng.standard_normal((N, n_q_cols))
    Hv = _unit_rows(z @ R_h) * norms[:, None]
    t0 = T // 4
    n_total = N + T
    H = np.empty((n_total, d))
    H[:t0] = rng.standard_normal((t0, d))
    H[t0:t0 + N] = Hv
    H[t0 + N:] = rng.standard_normal((T - t0, d))
    P = np.arange(n_total, dtype=np.int32)
    cast = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(dtype).contiguous()
    return Image(H=cast(H), K=cast(K), Q=cast(Q), P=torch.from_numpy(P), n_total=n_total,
                 vis_start=t0, N=N)


def _mixture_latents(rng, N, d_k, n_blobs, frac_blob, frac_dup, sig_lo, sig_hi, dup_eps):
    """Blob tokens, near-duplicates of earlier tokens, and wide-background tokens."""
    n_dup = int(round(frac_dup * N))
    n_blob = int(round(frac_blob * N))
    n_bg = N - n_dup - n_blob
    centres = _unit_rows(rng.standard_normal((n_blobs, d_k)))
    sig = rng.uniform(sig_lo, sig_hi, size=n_blobs)
    zb, _ = _blob_latents(rng, n_blob, centres, sig)
    bg_centre = _unit_rows(rng.standard_normal((1, d_k)))
    zg, _ = _blob_latents(rng, n_bg, bg_centre, np.array([1.0]))
    base = np.concatenate([zb, zg], axis=0)
    kind = np.concatenate([np.zeros(n_blob, np.int8), np.full(n_bg, 2, np.int8)])
    src = rng.integers(0, base.shape[0], size=n_dup)
    zd = base[src] + rng.standard_normal((n_dup, d_k)) * (dup_eps / np.sqrt(d_k))
    z = np.concatenate([base, zd], axis=0)
    kind = np.concatenate([kind, np.ones(n_dup, np.int8)])
    src_full = np.concatenate([np.arange(base.shape[0]), src])
    perm = rng.permutation(N)
    return z[perm], kind[perm], src_full[perm], perm


# --------------------------------------------------------------------------
# the five workloads
# --------------------------------------------------------------------------

def tiny(seed: int = 0, N: int = 196, T: int = 16, n_blobs: int = 12, sigma: float = 0.15,
         lam: float = 0.3, d_c: float = 0.4) -> Workload:
    """1 image, fp32, hidden 896, 2 KV heads x 64: the case the oracle does in well under a second."""
    d, n_h, d_h = 896, 2, 64
    d_k = n_h * d_h
    rng = np.random.default_rng(seed)
    centres = _unit_rows(rng.standard_normal((n_blobs, d_k)))
    z, which = _blob_latents(rng, N, centres, np.full(n_blobs, sigma))
    norms = rng.lognormal(0.0, 0.5, size=N)
    img = _assemble(rng, z, norms, d, d_k, T, torch.float32, proj_seed=10_000 + seed)
    return Workload("tiny", [img], d, n_h, n_h, d_h, torch.float32, lam, d_c,
                    extra={"blob_of_token": which, "n_blobs": n_blobs})


def single_image(seed: int = 1, N: int = 7290, T: int = 64, n_blobs: int = 200,
                 lam: float = 0.5, d_c: float = 0.3, dtype=torch.bfloat16,
                 d: int = 3584, n_h: int = 4, d_h: int = 128, n_qh: int | None = None,
                 distinct_k_clu: bool = False) -> Workload:
    """LLaVA-OneVision-7B-shaped single image: 50 % blob tokens, 30 % near-duplicates, 20 % low-norm background.

    n_qh > n_h gives grouped-query shapes; distinct_k_clu adds a second key buffer (a fixed
    rotation of the keys standing in for rotary embedding) for the clustering stage."""
    d_k = n_h * d_h
    n_qh = n_qh or n_h
    rng = np.random.default_rng(seed)
    z, kind, _, _ = _mixture_latents(rng, N, d_k, n_blobs, 0.5, 0.3, 0.1, 0.3, 0.02)
    norms = rng.lognormal(0.0, 0.5, size=N)
    norms[kind == 2] *= 0.05
    img = _assemble(rng, z, norms, d, n_qh * d_h, T, dtype, proj_seed=10_000 + seed)
    if distinct_k_clu:
        rot, _ = np.linalg.qr(np.random.default_rng(20_000 + seed).standard_normal((d_k, d_k)))
        img.K_clu = (img.K.to(torch.float64) @ torch.from_numpy(rot)).to(dtype).contiguous()
    return Workload("single_image", [img], d, n_qh, n_h, d_h, dtype, lam, d_c,
                    extra={"kind": kind})


def batched(seed: int = 2, B: int = 16, N: int = 2916, T: int = 32, lam: float = 0.5,
            d_c: float = 0.3, dtype=torch.bfloat16, d: int = 3584, n_h: int = 4,
            d_h: int = 128) -> Workload:
    """B independent images; the number of blobs per image is uniform in [50, 400]."""
    d_k = n_h * d_h
    rng = np.random.default_rng(seed)
    imgs, blobs = [], []
    for b in range(B):
        nb = int(rng.integers(50, 401))
        blobs.append(nb)
        z, kind, _, _ = _mixture_latents(rng, N, d_k, nb, 0.5, 0.3, 0.1, 0.3, 0.02)
        norms = rng.lognormal(0.0, 0.5, size=N)
        norms[kind == 2] *= 0.05
        imgs.append(_assemble(rng, z, norms, d, d_k, T, dtype, proj_seed=10_000 + seed))
    return Workload("batched", imgs, d, n_h, n_h, d_h, dtype, lam, d_c, extra={"blobs": blobs})


def video(seed: int = 3, frames: int = 32, per_frame: int = 196, T: int = 64, n_blobs: int = 40,
          sigma: float = 0.15, step: float = 0.05, redraw: float = 0.10, lam: float = 0.5,
          d_c: float = 0.3, dtype=torch.bfloat16, d: int = 3584, n_h: int = 4,
          d_h: int = 128) -> Workload:
    """Frame t is frame t-1 plus radius-`step` noise, with `redraw` of the positions resampled."""
    d_k = n_h * d_h
    rng = np.random.default_rng(seed)
    centres = _unit_rows(rng.standard_normal((n_blobs, d_k)))
    sig = np.full(n_blobs, sigma)
    cur, _ = _blob_latents(rng, per_frame, centres, sig)
    zs = [cur]
    for _ in range(1, frames):
        nxt = cur + rng.standard_normal(cur.shape) * (step / np.sqrt(d_k))
        moved = rng.random(per_frame) < redraw
        fresh, _ = _blob_latents(rng, int(moved.sum()), centres, sig)
        nxt[moved] = fresh
        zs.append(nxt)
        cur = nxt
    z = np.concatenate(zs, axis=0)
    norms = rng.lognormal(0.0, 0.5, size=z.shape[0])
    img = _assemble(rng, z, norms, d, d_k, T, dtype, proj_seed=10_000 + seed)
    return Workload("video", [img], d, n_h, n_h, d_h, dtype, lam, d_c)


def stress(seed: int = 4, B: int = 4, N: int = 16384, T: int = 64, n_blobs: int = 1000,
           lam: float = 0.7, d_c: float = 0.25, dup_frac: float = 0.01, dtype=torch.bfloat16,
           d: int = 3584, n_h: int = 4, d_h: int = 128) -> Workload:
    """Heavy-tailed norms, many blobs of variable spread, and 1 % exact duplicate tokens (density ties)."""
    d_k = n_h * d_h
    rng = np.random.default_rng(seed)
    imgs = []
    for b in range(B):
        centres = _unit_rows(rng.standard_normal((n_blobs, d_k)))
        sig = rng.uniform(0.05, 0.5, size=n_blobs)
        z, _ = _blob_latents(rng, N, centres, sig)
        norms = np.abs(rng.standard_t(3, size=N)) + 0.01
        img = _assemble(rng, z, norms, d, d_k, T, dtype, proj_seed=10_000 + seed)
        n_dup = int(round(dup_frac * N))
        dst = rng.choice(N, size=n_dup, replace=False)
        src = rng.integers(0, N, size=n_dup)
        keep = ~np.isin(src, dst)            # copy only from rows that are not overwritten themselves
        dst_t = torch.from_numpy(dst[keep])
        src_t = torch.from_numpy(src[keep])
        img.K[dst_t] = img.K[src_t]
        img.Q[dst_t] = img.Q[src_t]
        img.H[img.vis_start + dst_t] = img.H[img.vis_start + src_t]
        imgs.append(img)
    return Workload("stress", imgs, d, n_h, n_h, d_h, dtype, lam, d_c)


def layer_keys(seed: int = 5, n_layers: int = 10, N: int = 7290, n_h: int = 4, d_h: int = 128,
               dtype=torch.bfloat16, mix=None) -> List[torch.Tensor]:
    """Keys of the visual tokens at the first `n_layers` decoder layers, for the choice of the
    reduction layer: K_l[i] = gain_i * (shared_l + mix[l] * token_i,l) with a unit shared direction per
    layer and unit-scale token-specific noise.  With a small mix the keys of a layer are nearly
    parallel, as the first layers of the paper's model are described; the default mix grows with
    depth but not monotonically, so that "earliest layer above a threshold" and "layer with the
    widest keys" differ."""
    rng = np.random.default_rng(seed)
    d_k = n_h * d_h
    if mix is None:
        base = [0.02, 0.05, 0.04, 0.15, 0.4, 0.3, 0.9, 0.7, 1.5, 1.2]
        mix = [base[l % len(base)] for l in range(n_layers)]
    out = []
    for l in range(n_layers):
        shared = _unit_rows(rng.standard_normal((1, d_k)))
        tok = rng.standard_normal((N, d_k)) / np.sqrt(d_k)
        gain = rng.lognormal(0.0, 0.25, (N, 1))
        out.append(torch.from_numpy(gain * (shared + mix[l] * tok)).to(dtype).contiguous())
    return out


BUILDERS = {"tiny": tiny, "single_image": single_image, "batched": batched, "video": video,
            "stress": stress}


def build(name: str, **kw) -> Workload:
    return BUILDERS[name](**kw)
