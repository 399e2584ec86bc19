"""Pins for the CPU oracle: closed forms, hand-worked fixtures, brute force on tiny inputs,
the guarantees of Appendix B and degenerate cases.  None of these re-type the oracle's own
formulae with the same library call; each is chosen so that a dropped term, a wrong sign or
index, a wrong axis or a wrong inequality fails at least one of them."""
import itertools
import math
import os

import numpy as np
import pytest
import scipy.special

from oracle import pact_oracle as orc
from paper_2504_08966_b200 import workloads
from tests.helpers import f64, oracle_image

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed=0):
    return np.random.default_rng(seed)


# ------------------------------------------------------------------ EUTI (Eq. 1-4)

def test_euti_hand_example():
    want = None
    for line in open(os.path.join(GOLDEN, "euti_two_tokens.txt")):
        if line.startswith("scores"):
            want = [float(x) for x in line.split()[1:]]
    K = np.array([[math.log(3.0)], [0.0]])
    Q = np.array([[1.0], [1.0]])
    H = np.array([[3.0, 4.0], [0.0, 2.0]])
    s = orc.importance_scores(H, K, Q, 1, 1)
    assert np.allclose(s, want, rtol=1e-14)


def test_global_query_is_mean_over_tokens():
    Q = np.zeros((5, 2, 3))
    Q[:, 0, 1] = [1, 2, 3, 4, 5]
    Q[:, 1, 2] = 7
    g = orc.global_query(Q)
    assert g.shape == (2, 3) and g[0, 1] == 3.0 and g[1, 2] == 7.0 and g.sum() == 10.0


def test_scores_over_norm_sum_to_one():
    r = _rng(1)
    N, nh, dh, d = 50, 3, 8, 20
    H, K, Q = r.standard_normal((N, d)), r.standard_normal((N, nh * dh)), r.standard_normal((N, nh * dh))
    s = orc.importance_scores(H, K, Q, nh, nh)
    assert abs((s / np.linalg.norm(H, axis=1)).sum() - 1.0) < 1e-12


def test_zero_query_gives_norm_over_N():
    r = _rng(2)
    N, nh, dh, d = 17, 2, 4, 9
    H, K = r.standard_normal((N, d)), r.standard_normal((N, nh * dh))
    s = orc.importance_scores(H, K, np.zeros((N, nh * dh)), nh, nh)
    assert np.allclose(s, np.linalg.norm(H, axis=1) / N, rtol=1e-13)
    s2 = orc.importance_scores(H, np.tile(K[:1], (N, 1)), r.standard_normal((N, nh * dh)), nh, nh)
    assert np.allclose(s2, np.linalg.norm(H, axis=1) / N, rtol=1e-12)


def test_scores_match_independent_loops_with_gqa():
    """Per-head softmax over tokens, written as explicit loops with scipy's softmax, GQA 4 -> 2."""
    r = _rng(3)
    N, nq, nkv, dh, d = 9, 4, 2, 3, 5
    H, K, Q = r.standard_normal((N, d)), r.standard_normal((N, nkv * dh)), r.standard_normal((N, nq * dh))
    want = np.zeros(N)
    for j in range(nq):
        qg = [sum(Q[i, j * dh + t] for i in range(N)) / N for t in range(dh)]
        kv = j // (nq // nkv)
        logits = [sum(K[i, kv * dh + t] * qg[t] for t in range(dh)) for i in range(N)]
        want += scipy.special.softmax(np.array(logits))
    want = want / nq * np.array([math.sqrt(sum(x * x for x in H[i])) for i in range(N)])
    assert np.allclose(orc.importance_scores(H, K, Q, nq, nkv), want, rtol=1e-12)


def test_scores_invariant_to_key_shift_along_head():
    """Adding one vector to every key of a head shifts that head's logits by a constant."""
    r = _rng(4)
    N, nh, dh, d = 12, 2, 4, 6
    H, K, Q = r.standard_normal((N, d)), r.standard_normal((N, nh * dh)), r.standard_normal((N, nh * dh))
    K2 = K.copy()
    K2[:, :dh] += r.standard_normal(dh)
    assert np.allclose(orc.importance_scores(H, K, Q, nh, nh), orc.importance_scores(H, K2, Q, nh, nh), rtol=1e-10)


def test_score_ablations():
    r = _rng(5)
    N, nh, dh, d = 10, 2, 4, 6
    H, K, Q = r.standard_normal((N, d)), r.standard_normal((N, nh * dh)), r.standard_normal((N, nh * dh))
    full = orc.importance_scores(H, K, Q, nh, nh)
    no_norm = orc.importance_scores(H, K, Q, nh, nh, use_norm=False)
    norm_only = orc.importance_scores(H, K, Q, nh, nh, use_query=False)
    assert np.allclose(no_norm * np.linalg.norm(H, axis=1), full)
    assert abs(no_norm.sum() - 1) < 1e-12
    assert np.allclose(norm_only, np.linalg.norm(H, axis=1) / N)


@pytest.mark.parametrize("N", [1, 2, 5, 16])
def test_split_bruteforce(N):
    r = _rng(N)
    for lam in [0.0, 0.1, 0.3, 0.5, 0.99, 1.0]:
        s = r.random(N).astype(np.float32)
        if N > 3:
            s[1] = s[3]                                   # a tie
        tau, keep, kept, pruned = orc.split(s, lam)
        m = min(int(math.floor(lam * N + 1e-6)), N - 1)
        srt = sorted(float(x) for x in s)
        assert float(tau) == srt[m]
        assert [i for i in range(N) if s[i] >= tau] == list(kept)
        assert [i for i in range(N) if s[i] < tau] == list(pruned)
        assert len(pruned) <= m and len(kept) >= 1 and len(kept) + len(pruned) == N
        if lam == 0.0:
            assert keep.all()


def test_split_monotone_in_lambda_and_ties_kept():
    s = np.array([5, 1, 3, 3, 3, 9, 0], dtype=np.float32)
    prev = None
    for lam in np.linspace(0, 1, 15):
        _, keep, _, _ = orc.split(s, lam)
        if prev is not None:
            assert not (keep & ~prev).any()               # the kept set only shrinks
        prev = keep
    _, keep, _, pruned = orc.split(s, 3 / 7)              # m = 3 -> tau = 3, all three 3's stay
    assert list(pruned) == [1, 6] and keep[[2, 3, 4]].all()


# ------------------------------------------------------------------ distance, density (Eq. 5-6)

def test_distance_special_cases():
    U = np.array([[1.0, 0, 0], [0, 2.0, 0], [-3.0, 0, 0], [4.0, 0, 0], [1.0, math.sqrt(3.0), 0], [0, 0, 0]])
    D = orc.cosine_distance(U)
    assert D[0, 1] == 1.0 and D[0, 2] == 2.0 and D[0, 3] == 0.0
    assert abs(D[0, 4] - 0.5) < 1e-15                     # 60 degrees
    assert np.all(D[5, :5] == 1.0) and D[5, 5] == 0.0     # zero vector
    assert np.array_equal(D, D.T) and np.all(np.diag(D) == 0)
    assert D.min() >= 0 and D.max() <= 2


def test_distance_scale_invariant_and_rectangular_consistent():
    r = _rng(6)
    U = r.standard_normal((20, 7))
    s = 2.0 ** r.integers(-3, 4, size=20)
    assert np.array_equal(orc.cosine_distance(U), orc.cosine_distance(U * s[:, None]))
    D = orc.cosine_distance(U)
    R = orc.cosine_distance(U[:5], U[5:])
    assert np.allclose(R, D[:5, 5:], atol=1e-15)
    for i, j in [(0, 7), (3, 19)]:
        want = 1 - sum(U[i] * U[j]) / math.sqrt(sum(U[i] ** 2)) / math.sqrt(sum(U[j] ** 2))
        assert abs(D[i, j] - want) < 1e-14


def test_density_closed_forms():
    D = np.array([[0.0, 1.0], [1.0, 0.0]])
    assert np.allclose(orc.density(D, 2.0), 1 + math.exp(-0.5))
    r = _rng(7)
    U = r.standard_normal((30, 5))
    D = orc.cosine_distance(U)
    for dn in (0.5, 2.0):
        rho = orc.density(D, dn)
        assert np.all(rho <= 30) and np.all(rho >= 30 * math.exp(-2 / dn))
        assert abs(rho[4] - sum(math.exp(-D[4, j] / dn) for j in range(30))) < 1e-12


def test_duplicate_rows_have_equal_density_and_order_by_index():
    r = _rng(8)
    U = r.standard_normal((300, 64))
    U[257] = U[11]
    U[40] = U[199]
    D = orc.cosine_distance(U)
    rho = orc.density(D, 2.0)
    assert rho[257] == rho[11] and rho[40] == rho[199]
    order = list(orc.density_order(rho))
    assert order.index(11) + 1 == order.index(257) and order.index(40) + 1 == order.index(199)
    assert np.all(np.diff(rho[order]) <= 0)
    assert list(orc.density_order(np.array([1.0, 3.0, 3.0, 2.0, 3.0]))) == [1, 2, 4, 3, 0]


# ------------------------------------------------------------------ centres (Algorithm 2 / 4)

def _greedy_by_definition(D, rho, d_c):
    """Literal definition with explicit loops: process by (rho desc, index asc)."""
    q = len(rho)
    order = sorted(range(q), key=lambda i: (-rho[i], i))
    centres = []
    for i in order:
        if all(D[i][s] > d_c for s in centres):
            centres.append(i)
    return sorted(centres)


def test_two_arcs_fixture():
    angles, dn, cases = None, None, []
    for line in open(os.path.join(GOLDEN, "dbdpc_two_arcs.txt")):
        w = line.split()
        if not w or w[0].startswith("#"):
            continue
        if w[0] == "angles":
            angles = [float(x) for x in w[1:]]
        elif w[0] == "d_n":
            dn = float(w[1])
        elif w[0] == "case":
            ic, il = w.index("centres"), w.index("labels")
            cases.append((float(w[1]), [int(x) for x in w[ic + 1:il]], [int(x) for x in w[il + 1:]]))
    U = np.array([[math.cos(math.radians(a)), math.sin(math.radians(a))] for a in angles])
    assert len(cases) == 3
    for d_c, centres, labels in cases:
        out = orc.dbdpc(U, d_c, dn)
        assert list(out["centers"]) == centres
        assert list(out["label"]) == labels
        assert list(out["order"][:2]) == [1, 4]


@pytest.mark.parametrize("seed", range(6))
def test_centres_bruteforce_and_recursive_agree(seed):
    r = _rng(100 + seed)
    q = int(r.integers(2, 11))
    U = r.standard_normal((q, 3))
    if seed % 2:
        U[q - 1] = U[0]
    D = orc.cosine_distance(U)
    rho = orc.density(D, 2.0)
    order = orc.density_order(rho)
    for d_c in (0.0, 0.05, 0.3, 0.8, 1.5, 2.0):
        want = _greedy_by_definition(D.tolist(), rho.tolist(), d_c)
        assert list(orc.centers_sequential(D, order, d_c)) == want
        for T in (1, 3, 10 ** 9):
            assert list(orc.centers_recursive(D, order, d_c, T)) == want


@pytest.mark.parametrize("d_c", [0.05, 0.2, 0.5, 0.9])
def test_centre_guarantees_appendix_b(d_c):
    r = _rng(9)
    centres = r.standard_normal((15, 24))
    U = centres[r.integers(0, 15, 400)] + 0.35 * r.standard_normal((400, 24))
    out = orc.dbdpc(U, d_c, 2.0)
    D, C, lab = out["D"], out["centers"], out["label"]
    assert list(orc.centers_recursive(D, out["order"], d_c, 1)) == list(C)
    assert list(orc.centers_recursive(D, out["order"], d_c, 10)) == list(C)
    sub = D[np.ix_(C, C)] + 10 * np.eye(len(C))
    assert sub.min() > d_c                                       # centres pairwise farther than d_c
    assert np.all(D[np.arange(400), C[lab]] <= d_c)              # members within d_c of their centre
    assert np.all(D[:, C].min(axis=1) <= d_c)                    # maximal: nobody could still be a centre
    assert np.all(lab[C] == np.arange(len(C)))                   # a centre belongs to its own cluster
    same = lab[:, None] == lab[None, :]
    assert D[same].max() <= 2 * d_c * (2 - d_c) + 1e-12          # same-cluster pairs, Appendix B
    assert np.array_equal(lab, np.array([min(range(len(C)), key=lambda c: (D[i, C[c]], c)) for i in range(400)]))
    assert out["order"][0] in C                                  # the densest vector is always a centre


def test_centres_degenerate_cutoffs():
    r = _rng(10)
    U = r.standard_normal((40, 6))
    out = orc.dbdpc(U, 2.0, 2.0)
    assert list(out["centers"]) == [int(np.argmax(out["rho"]))] and np.all(out["label"] == 0)
    out0 = orc.dbdpc(U, 0.0, 2.0)
    assert list(out0["centers"]) == list(range(40))              # d_c = 0, no duplicates: no merging
    U2 = np.concatenate([U, U[:3] * 4.0])                        # same directions: distance exactly 0
    out1 = orc.dbdpc(U2, 0.0, 2.0)
    assert len(out1["centers"]) == 40 and np.array_equal(out1["label"][40:], out1["label"][:3])
    assert set(out1["centers"]).isdisjoint({40, 41, 42})         # ties in density go to the lower index


def test_exact_dc_is_member_not_centre():
    U = np.array([[1.0, 0.0], [0.5, math.sqrt(3) / 2], [0.9999, 0.01]])
    D = orc.cosine_distance(U)
    rho = np.array([3.0, 1.0, 2.0])
    order = orc.density_order(rho)
    assert list(orc.centers_sequential(D, order, D[0, 1])) == [0]     # d == d_c is not ">"
    assert list(orc.centers_sequential(D, order, np.nextafter(D[0, 1], 0))) == [0, 1]


# ------------------------------------------------------------------ reincorporation, merge

def test_reincorporate_bruteforce_and_extremes():
    r = _rng(11)
    Kc, Up = r.standard_normal((6, 5)), r.standard_normal((25, 5))
    Kc[4] = Kc[2] * 2                                           # equidistant centres: lowest id wins
    alpha, d_c = 1.5, 0.4
    lab, dmin = orc.reincorporate(Kc, Up, alpha, d_c)
    t = float(np.float32(alpha) * np.float32(d_c))
    for i in range(25):
        ds = [1 - float(Up[i] @ Kc[c]) / math.sqrt(float(Up[i] @ Up[i]) * float(Kc[c] @ Kc[c])) for c in range(6)]
        best = min(range(6), key=lambda c: (round(ds[c], 13), c))
        assert abs(dmin[i] - ds[best]) < 1e-13
        assert lab[i] == (best if ds[best] < t else -1)
        assert lab[i] != 4
    assert np.all(orc.reincorporate(Kc, Up, 0.0, d_c)[0] == -1)          # alpha = 0: nobody rejoins
    assert np.all(orc.reincorporate(Kc, Up, 6.0, 0.5)[0] >= 0)           # threshold 3 > 2: all rejoin
    assert orc.reinc_threshold(1.5, 0.3) == float(np.float32(1.5) * np.float32(0.3))


def test_merge_mean_sizes_positions():
    H = np.arange(24, dtype=np.float64).reshape(6, 4)
    P = np.array([10, 11, 12, 13, 14, 15])
    label = np.array([0, 1, 0, -1, 1, 1])
    Hm, Pm, sz = orc.merge(H, label, 2, np.array([2, 4]), P)
    assert np.array_equal(Hm[0], (H[0] + H[2]) / 2) and np.array_equal(Hm[1], (H[1] + H[4] + H[5]) / 3)
    assert list(Pm) == [12, 14] and list(sz) == [2, 3]
    Hc, _, _ = orc.merge(H, label, 2, np.array([2, 4]), P, center_only=True)
    assert np.array_equal(Hc, H[[2, 4]])


def test_proportional_attention_bias_equals_copies():
    """Eq. 11: a key with weight w and bias log w acts like w identical keys."""
    r = _rng(12)
    q, keys, vals = r.standard_normal(4), r.standard_normal((3, 4)), r.standard_normal((3, 2))
    sizes = np.array([1, 3, 2])
    a = scipy.special.softmax(keys @ q / 2.0 + orc.proportional_attention_bias(sizes)) @ vals
    rep = np.repeat(np.arange(3), sizes)
    b = scipy.special.softmax(keys[rep] @ q / 2.0) @ vals[rep]
    assert np.allclose(a, b, atol=1e-14)


# ------------------------------------------------------------------ choice of the layer L

def test_max_key_distance_closed_forms():
    """Known angles in the plane: the largest distance is 1 - cos of the widest angle."""
    ang = np.deg2rad([0.0, 20.0, 75.0, 130.0])
    K = np.stack([np.cos(ang), np.sin(ang)], axis=1) * np.array([[1.0], [7.0], [0.25], [3.0]])
    assert abs(orc.max_key_distance(K) - (1.0 - math.cos(math.radians(130.0)))) < 1e-14
    assert orc.max_key_distance(np.eye(5)) == 1.0                       # orthogonal keys
    assert orc.max_key_distance(np.array([[1.0, 2.0], [-2.0, -4.0]])) == 2.0   # opposite keys
    assert orc.max_key_distance(np.tile([[0.3, -1.0, 2.0]], (6, 1))) == 0.0    # identical keys
    assert orc.max_key_distance(np.array([[5.0, 1.0]])) == 0.0                 # one key


def test_max_key_distance_brute_force_and_scale_invariance():
    r = _rng(21)
    K = r.standard_normal((23, 7))
    best = 0.0
    for i, j in itertools.combinations(range(23), 2):
        c = sum(K[i, t] * K[j, t] for t in range(7)) / math.sqrt(sum(x * x for x in K[i]) * sum(x * x for x in K[j]))
        best = max(best, 1.0 - c)
    assert abs(orc.max_key_distance(K) - best) < 1e-13
    assert abs(orc.max_key_distance(K * r.uniform(0.1, 9.0, (23, 1))) - best) < 1e-13
    assert abs(orc.max_key_distance(K[r.permutation(23)]) - best) < 1e-13


def test_select_layer_takes_the_earliest_qualifying_layer():
    def fan(deg, n=9):
        a = np.deg2rad(np.linspace(0.0, deg, n))
        return np.stack([np.cos(a), np.sin(a)], axis=1)
    layers = [fan(10), fan(25), fan(60), fan(120), fan(40)]
    spreads = [1.0 - math.cos(math.radians(x)) for x in (10, 25, 60, 120, 40)]
    assert np.allclose([orc.max_key_distance(K) for K in layers], spreads, atol=1e-14)
    assert orc.select_layer(layers, 0.4) == 2            # 1 - cos 60 = 0.5 is the first >= 0.4
    assert orc.select_layer(layers, 0.5 - 1e-12) == 2 and orc.select_layer(layers, 0.5 + 1e-9) == 3
    assert orc.select_layer(layers, 0.0) == 0
    assert orc.select_layer(layers, 1.6) == -1
    assert orc.select_layer(layers[::-1], 0.2) == 0      # order matters: earliest, not largest


# ------------------------------------------------------------------ the whole step (Algorithm 3)

@pytest.fixture(scope="module")
def tiny_run():
    wl = workloads.tiny()
    return wl, wl.images[0], oracle_image(wl, wl.images[0])


def test_tiny_conservation_and_layout(tiny_run):
    wl, img, o = tiny_run
    N = img.N
    assert o["q"] + o["r"] + o["discarded"] == N
    assert o["size_out"][img.vis_start:img.vis_start + o["C"]].sum() == o["q"] + o["r"]
    assert o["n_out"] == o["C"] + (img.n_total - N) == o["H_out"].shape[0]
    H = f64(img.H)
    assert np.array_equal(o["H_out"][:img.vis_start], H[:img.vis_start])
    assert np.array_equal(o["H_out"][img.vis_start + o["C"]:], H[img.vis_start + N:])
    assert set(o["P_out"]) <= set(img.P.numpy()) and np.all(np.diff(o["P_out"]) > 0)
    assert np.array_equal(o["P_out"][img.vis_start:img.vis_start + o["C"]], img.P.numpy()[img.vis_start + o["center_idx"]])
    assert len(o["pruned_idx"]) <= orc.n_pruned(wl.lam, N)
    single = np.nonzero(o["size_out"][img.vis_start:img.vis_start + o["C"]] == 1)[0]
    for c in single:
        assert np.array_equal(o["H_out"][img.vis_start + c], H[img.vis_start + o["center_idx"][c]])
    t = orc.reinc_threshold(wl.alpha, wl.d_c)
    joined = o["label"][o["pruned_idx"]] >= 0
    assert np.all(o["dmin_pruned"][joined] < t) and np.all(o["dmin_pruned"][~joined] >= t)


def test_tiny_recovers_planted_blobs(tiny_run):
    wl, img, o = tiny_run
    blob = wl.extra["blob_of_token"]
    kept = o["kept_idx"]
    assert o["C"] == len(set(blob[kept]))
    lab = o["label"]
    for b in set(blob[kept]):
        assert len(set(lab[kept][blob[kept] == b])) == 1
    assert len(set(lab[kept])) == o["C"]
    joined = lab >= 0
    assert all(lab[i] == lab[kept][blob[kept] == blob[i]][0] for i in np.nonzero(joined)[0])


def test_lambda_zero_is_pure_dbdpc(tiny_run):
    wl, img, _ = tiny_run
    o = oracle_image(wl, img, lam=0.0)
    assert o["q"] == img.N and o["r"] == 0 and o["discarded"] == 0
    ref = orc.dbdpc(f64(img.K), wl.d_c, wl.d_n)
    assert np.array_equal(o["center_idx"], ref["centers"]) and np.array_equal(o["label"], ref["label"])


def test_alpha_zero_and_tiny_dc(tiny_run):
    wl, img, base = tiny_run
    o = oracle_image(wl, img, alpha=0.0)
    assert o["r"] == 0 and np.array_equal(o["center_idx"], base["center_idx"])
    o2 = oracle_image(wl, img, d_c=1e-9)
    assert o2["C"] == o2["q"] and o2["r"] == 0                    # d_c -> 0: no merging at all
    sl = slice(img.vis_start, img.vis_start + o2["C"])
    assert np.array_equal(o2["H_out"][sl], f64(img.H)[img.vis_start + o2["kept_idx"]])


def test_small_bf16_mixture_invariants():
    wl = workloads.single_image(seed=5, N=600, T=8, n_blobs=20, d=256, n_h=2, d_h=32)
    img = wl.images[0]
    o = oracle_image(wl, img)
    assert o["q"] + o["r"] + o["discarded"] == img.N
    D, C = o["D"], o["centers_local"]
    assert list(orc.centers_recursive(D, o["order"], float(np.float32(wl.d_c)), 10)) == list(C)
    assert 1 < o["C"] < o["q"]
    lk = o["label"][o["kept_idx"]]
    assert np.all(D[np.arange(o["q"]), C[lk]] <= np.float32(wl.d_c))


# ---- the split with a given number of pruned tokens, replay, fragile decisions, planted mistakes --------

@pytest.mark.parametrize("N", [1, 2, 7, 16])
def test_split_with_given_m_bruteforce(N):
    """split(s, lam, m) cuts the tokens strictly below the (m+1)-th smallest score, whatever lam says."""
    rng = np.random.default_rng(100 + N)
    s = rng.integers(0, 5, N).astype(np.float32)            # many ties
    for m in range(-1, N + 2):
        tau, keep, kept, pruned = orc.split(s, 0.9, m)
        mm = min(max(m, 0), N - 1)
        want_tau = sorted(s.tolist())[mm]
        assert tau == want_tau
        assert keep.tolist() == [x >= want_tau for x in s.tolist()]
        assert pruned.size <= mm and kept.size + pruned.size == N
        assert kept.tolist() == sorted(kept.tolist()) and pruned.tolist() == sorted(pruned.tolist())
    # the derived m and the given m agree when they are the same number
    a = orc.split(s, 0.5)
    b = orc.split(s, 0.0, orc.n_pruned(0.5, N))
    assert a[0] == b[0] and np.array_equal(a[1], b[1])


def test_pact_reduce_with_given_m_equals_lambda_that_gives_it():
    wl = workloads.tiny()
    img = wl.images[0]
    m = orc.n_pruned(wl.lam, img.N)
    a = oracle_image(wl, img)
    b = oracle_image(wl, img, lam=0.0, n_prune=m)
    assert np.array_equal(a["keep"], b["keep"]) and np.array_equal(a["label"], b["label"])
    c = oracle_image(wl, img, n_prune=0)                    # nothing pruned
    assert c["q"] == img.N and c["r"] == 0


def test_replay_of_own_decisions_changes_nothing_and_a_given_order_is_followed():
    wl = workloads.tiny()
    img = wl.images[0]
    a = oracle_image(wl, img)
    b = oracle_image(wl, img, keep_given=a["keep"], order_given=a["order"])
    assert np.array_equal(a["label"], b["label"]) and np.array_equal(a["H_out"], b["H_out"])
    # a different keep mask is taken as given
    keep = a["keep"].copy()
    flip = int(np.nonzero(keep)[0][0])
    keep[flip] = False
    c = oracle_image(wl, img, keep_given=keep)
    assert c["q"] == a["q"] - 1 and not c["keep"][flip]
    # three collinear points 0 - 1 - 2 with d(0,1), d(1,2) <= d_c < d(0,2): the order decides the centres
    ang = np.array([0.0, 0.5, 1.0])
    U = np.stack([np.cos(ang), np.sin(ang)], axis=1)
    d_c = 1 - math.cos(0.6)
    assert orc.dbdpc(U, d_c, 2.0, order=np.array([1, 0, 2]))["centers"].tolist() == [1]
    assert orc.dbdpc(U, d_c, 2.0, order=np.array([0, 1, 2]))["centers"].tolist() == [0, 2]


def test_fragile_decisions_on_a_hand_made_case():
    """Every class is planted once and must be counted once."""
    scores = np.array([1.0, 2.0, 2.0 + 1e-6, 3.0, 2.0])     # tau = 2: one score within 1e-6 tau above it
    d_c = 0.5
    D = np.array([[0.0, 0.5 + 5e-7, 0.9], [0.5 + 5e-7, 0.0, 0.2], [0.9, 0.2, 0.0]])   # pair (0,1) in the d_c band
    rho = np.array([2.0, 3.0, 3.0 - 1e-6])                  # 1 and 2 are neighbours in the order, within d_c
    order = np.array([1, 2, 0])
    Dk = np.array([[0.1, 0.1 + 5e-7], [0.0, 0.7], [0.7, 0.0]])   # row 0: two centres within 1e-6
    Dp = np.array([[0.75 - 2e-7, 1.0], [0.3, 0.9]])         # row 0: nearest centre within 1e-6 of alpha d_c = 0.75
    f = orc.fragile_decisions(scores, 2.0, D, rho, order, d_c, Dk, Dp, 0.75)
    assert (f["score_tau"], f["rho_order"], f["band_dc"], f["band_adc"], f["argmin"]) == (1, 1, 1, 1, 1)
    assert abs(f["score_tau_min_rel"] - 5e-7) < 1e-9 and abs(f["band_dc_min"] - 5e-7) < 1e-12
    # moved away by ten times the tolerance, nothing is counted
    D2 = D.copy(); D2[0, 1] = D2[1, 0] = 0.5 + 1e-5
    f2 = orc.fragile_decisions(np.array([1.0, 2.0, 2.1, 3.0, 2.0]), 2.0, D2, np.array([2.0, 3.0, 2.9]), order, d_c,
                               np.array([[0.1, 0.2], [0.0, 0.7], [0.7, 0.0]]), np.array([[0.7, 1.0], [0.3, 0.9]]), 0.75)
    assert (f2["score_tau"], f2["rho_order"], f2["band_dc"], f2["band_adc"], f2["argmin"]) == (0, 0, 0, 0, 0)


def _mutants():
    """Plausible slips, each planted in a copy of one oracle function (on the CPU, never in the product)."""
    real_distance = orc.cosine_distance
    def dist_wrong_sign(U, V=None):
        D = real_distance(U, V)
        return np.clip(2.0 - D, 0.0, 2.0) if V is None else 2.0 - D          # 1 + cos instead of 1 - cos
    def density_without_self(D, d_n):
        return np.exp(-D / d_n).sum(axis=1) - 1.0                               # dropped j = i
    def order_ascending(rho):
        return np.argsort(rho, kind="stable")                                   # sorted the wrong way
    def centres_not_strict(D, order, d_c):
        centers = []
        for i in order:
            if not centers or D[i, centers].min() >= d_c:                       # >= instead of >
                centers.append(int(i))
        return np.array(sorted(centers), dtype=np.int64)
    def scores_softmax_over_heads(H, K, Q, n_qh, n_kvh, use_norm=True, use_query=True):
        N = H.shape[0]; d_h = K.shape[1] // n_kvh
        Kd = K.astype(np.float64).reshape(N, n_kvh, d_h); Qg = orc.global_query(Q.astype(np.float64).reshape(N, n_qh, d_h))
        L = np.stack([Kd[:, (j * n_kvh) // n_qh, :] @ Qg[j] for j in range(n_qh)], axis=1)
        P = np.exp(L - L.max(axis=1, keepdims=True)); P /= P.sum(axis=1, keepdims=True)   # softmax over the wrong axis
        return P.mean(axis=1) * np.sqrt((H.astype(np.float64) ** 2).sum(axis=1))
    return {"cosine_distance": dist_wrong_sign, "density": density_without_self, "density_order": order_ascending,
            "centers_sequential": centres_not_strict, "importance_scores": scores_softmax_over_heads}


@pytest.mark.parametrize("name", ["cosine_distance", "density", "density_order", "centers_sequential", "importance_scores"])
def test_a_planted_mistake_fails_a_pin(name, monkeypatch):
    """The pins are only worth something if a wrong oracle fails them: plant one mistake at a time."""
    pins = {"cosine_distance": test_distance_special_cases, "density": test_density_closed_forms,
            "density_order": test_duplicate_rows_have_equal_density_and_order_by_index,
            "centers_sequential": test_exact_dc_is_member_not_centre, "importance_scores": test_scores_over_norm_sum_to_one}
    pins[name]()                                            # green with the real function
    monkeypatch.setattr(orc, name, _mutants()[name])
    with pytest.raises(AssertionError):
        pins[name]()
