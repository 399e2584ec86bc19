"""CPU oracle for PACT's visual-token reduction step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, float64 restatement of what the paper defines, written from the
paper and sharing no code with the CUDA path.  Only the tests, the smoke check
and the benchmark's CPU-baseline leg may import it; the product never does.

Steps and the passages they follow
----------------------------------
* ``global_query``        Eq. 1 / Algorithm 1 step 1
* ``importance_scores``   Eq. 2 / Algorithm 1 step 2 (softmax across visual tokens, per head)
* ``split``               Eq. 3-4 / Algorithm 1 step 3
* ``cosine_distance``     Eq. 5
* ``density``             Eq. 6
* ``density_order``       Algorithm 2 ("sort by rho, descending"); tie rule of Appendix D.1
* ``centers_sequential``  Algorithm 2, the centre loop (this DEFINES the result)
* ``centers_recursive``   Algorithm 4 (written separately; must give the same set, Appendix D.2)
* ``nearest_center``      Algorithm 2, the assignment loop
* ``reincorporate``       Eq. 8-9 / Algorithm 3 step 3
* ``merge``               Eq. 10 / Algorithm 3 step 4 (mean of members; centre's position id)
* ``proportional_attention_bias``  Eq. 11 (log of the cluster sizes)
* ``max_key_distance``, ``select_layer``  choice of the reduction layer L (the paragraph after
  Eq. 11 and the figure it refers to: largest distance between two visual keys of a layer;
  the earliest layer where it is high enough)
* ``pact_reduce``         Algorithm 3 end to end (with a replay mode for the keep mask and the density order)
* ``fragile_decisions``   counts, in float64, of the real-valued comparisons that sit within 1e-6 of turning

Readings taken where the paper is silent or garbled (each is also listed in the
design notes): softmax runs over the visual tokens separately per head and
without a 1/sqrt(d_h) factor; Percentile(s, lambda) is the order statistic
with m = min(floor(lambda*N + 1e-6), N-1) tokens strictly below it; scores
are float32 quantities (the library returns them as such) and the split is
taken on those float32 values; the clustering vector of a token is the
concatenation of its key heads; a zero key has distance 1 to everything;
d_ii = 0; density ties go to the lower token index; a centre needs distance
strictly greater than d_c to every earlier centre; argmin ties go to the
centre with the lowest token index; cluster ids number the centres by
ascending token index; reincorporation needs distance strictly below
float32(alpha)*float32(d_c); the distance between keys that decides the layer is
the cosine distance of Eq. 5 on the full key vectors, "sufficiently high" is
>= a threshold the caller gives, and no layer qualifying is reported as -1.

Pins: every function here is pinned by tests/test_oracle_pins.py against closed
forms, brute force on tiny inputs, invariants of Appendix B and degenerate
cases.  The paper prints no worked numeric example, so there is no golden
vector from the paper itself.
"""
from __future__ import annotations

import numpy as np

_TINY_NORM = 1e-20


# --------------------------------------------------------------------------
# EUTI (Algorithm 1)
# --------------------------------------------------------------------------

def global_query(Q: np.ndarray) -> np.ndarray:
    """Eq. 1: mean of the query vectors over the visual tokens.  Q is [N, n_qh, d_h]."""
    return Q.astype(np.float64).sum(axis=0) / Q.shape[0]


def importance_scores(H: np.ndarray, K: np.ndarray, Q: np.ndarray, n_qh: int, n_kvh: int,
                      use_norm: bool = True, use_query: bool = True) -> np.ndarray:
    """Eq. 2.  H [N, d], K [N, n_kvh*d_h], Q [N, n_qh*d_h] -> float64 scores [N].

    Query head j is paired with key head floor(j * n_kvh / n_qh) (grouped-query
    attention; with n_qh == n_kvh this is the paper's literal statement).
    ``use_norm`` / ``use_query`` switch off one factor (the ablations of Sec. 4).
    """
    N = H.shape[0]
    d_h = K.shape[1] // n_kvh
    Hd = H.astype(np.float64)
    Kd = K.astype(np.float64).reshape(N, n_kvh, d_h)
    Qd = Q.astype(np.float64).reshape(N, n_qh, d_h)
    Qg = global_query(Qd)                                   # [n_qh, d_h]
    p_mean = np.zeros(N)
    for j in range(n_qh):
        kv = (j * n_kvh) // n_qh
        logit = Kd[:, kv, :] @ Qg[j]                        # k_i^(j) . Qglobal^(j)
        e = np.exp(logit - logit.max())
        p_mean += e / e.sum()                               # softmax across visual tokens
    p_mean /= n_qh
    if not use_query:
        p_mean = np.full(N, 1.0 / N)
    norm = np.sqrt((Hd * Hd).sum(axis=1)) if use_norm else np.ones(N)
    return p_mean * norm


def n_pruned(lam: float, N: int) -> int:
    """Number of tokens the percentile aims to cut: min(floor(lambda*N + 1e-6), N-1)."""
    return int(min(np.floor(float(lam) * N + 1e-6), N - 1))


def split(scores32: np.ndarray, lam: float, m: int | None = None):
    """Eq. 3-4 on float32 scores.  Returns tau, keep mask, kept and pruned indices (ascending).
    m: the number of tokens the percentile aims to cut, given directly instead of through lambda
    (clamped to [0, N-1] like the derived one)."""
    s = np.asarray(scores32, dtype=np.float32)
    N = s.shape[0]
    m = n_pruned(lam, N) if m is None else int(min(max(int(m), 0), N - 1))
    tau = np.sort(s, kind="stable")[m]                      # (m+1)-th smallest score
    keep = s >= tau
    return tau, keep, np.nonzero(keep)[0].astype(np.int32), np.nonzero(~keep)[0].astype(np.int32)


# --------------------------------------------------------------------------
# DBDPC (Algorithm 2)
# --------------------------------------------------------------------------

def cosine_distance(U: np.ndarray, V: np.ndarray | None = None) -> np.ndarray:
    """Eq. 5: d = 1 - u.v / (|u||v|), clamped to [0, 2]; with V omitted, all pairs of U and d_ii = 0.

    |u||v| is formed as sqrt(|u|^2 |v|^2) so that two identical (or power-of-two scaled)
    vectors are at distance exactly 0 in floating point as they are in the mathematics."""
    Ud = U.astype(np.float64)
    nu2 = np.maximum((Ud * Ud).sum(axis=1), _TINY_NORM ** 2)
    if V is None:
        D = 1.0 - (Ud @ Ud.T) / np.sqrt(nu2[:, None] * nu2[None, :])
        D = np.clip(D, 0.0, 2.0)
        np.fill_diagonal(D, 0.0)
        return D
    Vd = V.astype(np.float64)
    nv2 = np.maximum((Vd * Vd).sum(axis=1), _TINY_NORM ** 2)
    return np.clip(1.0 - (Ud @ Vd.T) / np.sqrt(nu2[:, None] * nv2[None, :]), 0.0, 2.0)


def density(D: np.ndarray, d_n: float) -> np.ndarray:
    """Eq. 6: rho_i = sum_j exp(-d_ij / d_n), j over every vector including i."""
    return np.exp(-D / float(d_n)).sum(axis=1)


def density_order(rho: np.ndarray) -> np.ndarray:
    """Indices by descending density; equal densities keep ascending index order."""
    return np.argsort(-rho, kind="stable")


def centers_sequential(D: np.ndarray, order: np.ndarray, d_c: float) -> np.ndarray:
    """Algorithm 2's centre loop: visit in density order; a vector becomes a centre iff its
    smallest distance to the centres chosen so far is strictly greater than d_c."""
    centers = []
    for i in order:
        if not centers or D[i, centers].min() > d_c:
            centers.append(int(i))
    return np.array(sorted(centers), dtype=np.int64)


def centers_recursive(D: np.ndarray, order: np.ndarray, d_c: float, T: int = 10) -> np.ndarray:
    """Algorithm 4: rounds of "delta_i > d_c" over the live set with a sequential tail.

    delta_i is the smallest distance from i to a live vector of higher density
    (earlier in `order`), Eq. 12.  Vectors within d_c of a new centre leave the
    live set.  When a round finds fewer than T centres the remaining vectors are
    finished by the sequential rule against all centres found so far.
    """
    q = D.shape[0]
    rank = np.empty(q, dtype=np.int64)
    rank[order] = np.arange(q)
    live = np.ones(q, dtype=bool)
    centers: list[int] = []
    while live.any():
        idx = np.nonzero(live)[0]
        sub = D[np.ix_(idx, idx)]
        higher = rank[idx][None, :] < rank[idx][:, None]          # column has higher density than row
        delta = np.where(higher, sub, np.inf).min(axis=1)
        new = idx[delta > d_c]
        centers.extend(int(c) for c in new)
        live[new] = False
        if new.size:
            near = (D[:, new] <= d_c).any(axis=1)
            live &= ~near
        if new.size < T:
            rest = [i for i in order if live[i]]
            for i in rest:
                if not centers or D[i, centers].min() > d_c:
                    centers.append(int(i))
            break
    return np.array(sorted(centers), dtype=np.int64)


def nearest_center(Dc: np.ndarray):
    """Algorithm 2's assignment: argmin over centres (columns, already in ascending token
    index); numpy's argmin returns the first minimum, i.e. the lowest cluster id."""
    a = Dc.argmin(axis=1)
    return a.astype(np.int64), Dc[np.arange(Dc.shape[0]), a]


def dbdpc(U: np.ndarray, d_c: float, d_n: float, order: np.ndarray | None = None):
    """Algorithm 2 on the rows of U.  Returns a dict with D, rho, order, centres (ascending
    local indices) and the cluster id of every row.  order: replay a given density order
    instead of the one derived from rho (see pact_reduce)."""
    D = cosine_distance(U)
    rho = density(D, d_n)
    order = density_order(rho) if order is None else np.asarray(order, dtype=np.int64)
    centers = centers_sequential(D, order, float(np.float32(d_c)))
    label, dmin = nearest_center(D[:, centers])
    return {"D": D, "rho": rho, "order": order, "centers": centers, "label": label, "dmin": dmin}


# --------------------------------------------------------------------------
# reincorporation, merge (Algorithm 3 steps 3-4)
# --------------------------------------------------------------------------

def reinc_threshold(alpha: float, d_c: float) -> float:
    """float32(alpha) * float32(d_c), formed in float32 (both sides use this value)."""
    return float(np.float32(alpha) * np.float32(d_c))


def reincorporate(Kc: np.ndarray, U_pruned: np.ndarray, alpha: float, d_c: float):
    """Eq. 8: a pruned token joins its nearest centre iff that distance is < alpha*d_c.
    Kc: centre keys in cluster-id order.  Returns (cluster id or -1, nearest distance)."""
    if U_pruned.shape[0] == 0:
        return np.zeros(0, dtype=np.int64), np.zeros(0)
    Dp = cosine_distance(U_pruned, Kc)
    a, dmin = nearest_center(Dp)
    t = reinc_threshold(alpha, d_c)
    return np.where(dmin < t, a, -1), dmin


def merge(Hv: np.ndarray, label: np.ndarray, n_clusters: int, center_token: np.ndarray,
          Pv: np.ndarray, center_only: bool = False):
    """Eq. 10: mean of the members' hidden states per cluster; position id of the centre.
    label[i] = cluster id or -1 (discarded).  Returns (H' float64, P', sizes)."""
    Hd = Hv.astype(np.float64)
    Hout = np.zeros((n_clusters, Hd.shape[1]))
    sizes = np.zeros(n_clusters, dtype=np.int64)
    for c in range(n_clusters):
        members = np.nonzero(label == c)[0]
        sizes[c] = members.size
        Hout[c] = Hd[center_token[c]] if center_only else Hd[members].sum(axis=0) / members.size
    return Hout, Pv[center_token].copy(), sizes


def proportional_attention_bias(sizes: np.ndarray) -> np.ndarray:
    """Eq. 11: the additive logit bias log(w) of a merged token that stands for w tokens."""
    return np.log(sizes.astype(np.float64))


def max_key_distance(K: np.ndarray) -> float:
    """Largest distance (Eq. 5) between two of the visual keys of one layer; 0 for a single key."""
    return float(cosine_distance(K).max())


def select_layer(K_layers, threshold: float) -> int:
    """The earliest layer whose largest key distance is at least `threshold`; -1 if there is none."""
    for layer, K in enumerate(K_layers):
        if max_key_distance(K) >= threshold:
            return layer
    return -1


# --------------------------------------------------------------------------
# the whole step (Algorithm 3)
# --------------------------------------------------------------------------

def fragile_decisions(scores, tau, D, rho, order, d_c, Dk_centers, Dp_centers, t_reinc, tol=1e-6):
    """Real-valued decisions of one image that a different rounding could turn, counted in float64.

    Every discrete output hangs on comparisons of real numbers.  A pair within `tol` of d_c (or a
    pruned token within `tol` of alpha d_c) is the one class the specification exempts; the others are
    reported so that a mismatch can be traced to its root:
      score_tau   tokens whose score differs from tau but by at most tol * tau (Eq. 3-4)
      rho_order   neighbours in the density order whose densities differ by at most tol * rho and that
                  lie within d_c (1 + tol) of each other (only such a pair can change a centre)
      band_dc     unordered pairs of survivors with |d - d_c| <= tol (Algorithm 2's centre test)
      band_adc    pruned tokens whose nearest-centre distance is within tol of alpha d_c (Eq. 8)
      argmin      tokens whose two nearest centres differ by at most tol in distance (Algorithm 2's
                  assignment and Eq. 8's nearest centre)
    Each class comes with its smallest margin (None when the class has no candidate at all)."""
    s = np.asarray(scores, dtype=np.float64)
    tau = float(tau)
    ds = np.abs(s - tau)
    off = ds[ds > 0]
    out = {"score_tau": int(((ds > 0) & (ds <= tol * abs(tau))).sum()),
           "score_tau_min_rel": float(off.min() / abs(tau)) if off.size and tau != 0 else None}
    a, b = order[:-1], order[1:]
    gap = rho[a] - rho[b]
    near = D[a, b] <= d_c * (1 + tol)
    out["rho_order"] = int((near & (gap <= tol * rho[a])).sum())
    out["rho_order_min_rel"] = float((gap[near] / rho[a][near]).min()) if near.any() else None
    iu = np.triu_indices(D.shape[0], 1)
    dd = np.abs(D[iu] - d_c)
    out["band_dc"] = int((dd <= tol).sum())
    out["band_dc_min"] = float(dd.min()) if dd.size else None
    dp = np.abs(Dp_centers.min(axis=1) - t_reinc) if Dp_centers.shape[0] and Dp_centers.shape[1] else np.zeros(0)
    out["band_adc"] = int((dp <= tol).sum())
    out["band_adc_min"] = float(dp.min()) if dp.size else None
    n_close, min_gap = 0, None
    for Dc in (Dk_centers, Dp_centers):
        if Dc.shape[0] and Dc.shape[1] >= 2:
            two = np.partition(Dc, 1, axis=1)[:, :2]
            g = two[:, 1] - two[:, 0]
            n_close += int((g <= tol).sum())
            min_gap = float(g.min()) if min_gap is None else min(min_gap, float(g.min()))
    out["argmin"] = n_close
    out["argmin_min"] = min_gap
    return out


def pact_reduce(H, K_euti, Q_euti, K_clu, P, vis_start, N, n_qh, n_kvh, lam, d_c, d_n=2.0,
                alpha=1.5, use_norm=True, use_query=True, center_only=False, n_prune=None,
                keep_given=None, order_given=None):
    """Algorithm 3 on one image.  H [n_total, d], P [n_total]; K/Q rows are the N visual tokens.

    Returns every intermediate the parity tests compare, plus the near-threshold decisions of
    `fragile_decisions` under "fragile" (band_dc and band_adc also at the top level).

    Replay: keep_given (bool [N]) replaces the keep mask of Eq. 3-4 and order_given (survivor
    positions by descending density) replaces the density order of Algorithm 2, so that when one
    of those decisions was turned by a near-tie every later stage can still be compared exactly.
    """
    n_total = H.shape[0]
    Hv = H[vis_start:vis_start + N]
    scores = importance_scores(Hv, K_euti, Q_euti, n_qh, n_kvh, use_norm, use_query)
    scores32 = scores.astype(np.float32)
    tau, keep, kept, pruned = split(scores32, lam, n_prune)
    if keep_given is not None:
        keep = np.asarray(keep_given, dtype=bool)
        kept = np.nonzero(keep)[0].astype(np.int32)
        pruned = np.nonzero(~keep)[0].astype(np.int32)
    dc = float(np.float32(d_c))
    cl = dbdpc(K_clu[kept], dc, d_n, order_given)
    centers_local = cl["centers"]
    center_token = kept[centers_local].astype(np.int64)      # ascending token index = cluster id order
    C = center_token.size
    label = np.full(N, -1, dtype=np.int64)
    label[kept] = cl["label"]
    lab_p, dmin_p = reincorporate(K_clu[center_token], K_clu[pruned], alpha, dc)
    label[pruned] = lab_p
    Hm, Pm, sizes = merge(Hv, label, C, center_token, P[vis_start:vis_start + N], center_only)
    n_out = n_total - N + C
    H_out = np.concatenate([H[:vis_start].astype(np.float64), Hm,
                            H[vis_start + N:].astype(np.float64)], axis=0)
    P_out = np.concatenate([P[:vis_start], Pm, P[vis_start + N:]])
    size_out = np.concatenate([np.ones(vis_start, np.int64), sizes,
                               np.ones(n_total - vis_start - N, np.int64)])
    t = reinc_threshold(alpha, dc)
    Dp = cosine_distance(K_clu[pruned], K_clu[center_token]) if pruned.size else np.zeros((0, C))
    # the threshold in float64: the smallest float64 score that was kept (tau itself is a float32 value, which
    # differs from the float64 score of the token that defines it by its own rounding)
    tau64 = float(scores[keep].min()) if keep.any() else float(tau)
    frag = fragile_decisions(scores, tau64, cl["D"], cl["rho"], cl["order"], dc, cl["D"][:, centers_local], Dp, t)
    return {
        "scores": scores, "scores32": scores32, "tau": tau, "keep": keep, "kept_idx": kept,
        "pruned_idx": pruned, "D": cl["D"], "rho": cl["rho"], "order": cl["order"],
        "centers_local": centers_local, "center_idx": center_token, "label": label,
        "dmin_kept": cl["dmin"], "dmin_pruned": dmin_p,
        "H_out": H_out, "P_out": P_out, "size_out": size_out, "n_out": n_out,
        "logw_out": proportional_attention_bias(size_out),
        "q": int(kept.size), "C": int(C), "r": int((lab_p >= 0).sum()),
        "discarded": int((lab_p < 0).sum()),
        "band_dc": frag["band_dc"], "band_adc": frag["band_adc"], "fragile": frag,
    }
