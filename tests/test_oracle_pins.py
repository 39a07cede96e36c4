"""Pins for the CPU oracle: closed forms, brute force, invariants and the paper's printed numbers.

None of these tests touches the CUDA path; they establish that ``oracle/`` computes what the
paper defines before anything is compared against it.
"""
import itertools
import math
import os

import numpy as np
import pytest

import oracle
from paper_2601_17818_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16(x):
    return W.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


# =============================================================================== O1: K-norm (Eq. 4)
def test_knorm_constant_closed_form():
    # all entries c  ->  |c| * sqrt(H*d);  c = 1, H = 32, d = 128  ->  exactly 64
    K = bf16(np.ones((2, 32, 5, 128)))
    s = oracle.knorm(K, 0, 5)
    assert np.array_equal(s, np.full((2, 5), 64.0))
    K = bf16(np.full((1, 8, 3, 64), -0.5))
    assert np.array_equal(oracle.knorm(K, 0, 3), np.full((1, 3), 0.5 * math.sqrt(8 * 64)))


def test_knorm_one_hot_and_zero():
    K = np.zeros((1, 4, 6, 16), dtype=np.float32)
    K[0, 2, 3, 7] = -3.0
    K[0, 1, 4, 0] = 0.375
    s = oracle.knorm(bf16(K), 0, 6)[0]
    assert s[3] == 3.0 and s[4] == 0.375
    assert np.all(s[[0, 1, 2, 5]] == 0.0)


def test_knorm_equals_frobenius_norm_of_flattened_row():
    rng = np.random.default_rng(1)
    Kf = W.bf16_bits_to_f32(bf16(rng.standard_normal((3, 5, 11, 24))))
    s = oracle.knorm(bf16(Kf), 0, 11)
    flat = np.transpose(Kf.astype(np.float64), (0, 2, 1, 3)).reshape(3, 11, -1)
    ref = np.linalg.norm(flat, axis=-1)                 # textbook L2 norm of the concatenated heads
    np.testing.assert_allclose(s, ref, rtol=1e-14)


def test_knorm_span_and_invariances():
    rng = np.random.default_rng(2)
    Kf = W.bf16_bits_to_f32(bf16(rng.standard_normal((2, 6, 20, 16))))
    full = oracle.knorm(bf16(Kf), 0, 20)
    part = oracle.knorm(bf16(Kf), 7, 9)                 # only the visual span [7, 16) is scored
    assert np.array_equal(part, full[:, 7:16])
    ragged = oracle.knorm(bf16(Kf), 3, np.array([4, 10], dtype=np.int32))
    assert np.array_equal(ragged[0, :4], full[0, 3:7]) and np.array_equal(ragged[1], full[1, 3:13])
    # permuting heads or elements changes only the summation order
    perm_h = oracle.knorm(bf16(Kf[:, ::-1]), 0, 20)
    perm_e = oracle.knorm(bf16(Kf[..., ::-1]), 0, 20)
    np.testing.assert_allclose(perm_h, full, rtol=1e-14)
    np.testing.assert_allclose(perm_e, full, rtol=1e-14)
    # scaling by a power of two is exact
    assert np.array_equal(oracle.knorm(bf16(Kf * 8.0), 0, 20), full * 8.0)


def test_knorm_is_rotation_invariant():
    # rotating (e_2t, e_2t+1) pairs (RoPE) leaves the norm unchanged; done in float64 before
    # rounding is impossible in bf16, so check the identity on exactly representable rotations (90 degrees)
    rng = np.random.default_rng(3)
    Kf = W.bf16_bits_to_f32(bf16(rng.standard_normal((1, 2, 4, 8))))
    rot = np.empty_like(Kf)
    rot[..., 0::2] = -Kf[..., 1::2]
    rot[..., 1::2] = Kf[..., 0::2]
    np.testing.assert_allclose(oracle.knorm(bf16(rot), 0, 4), oracle.knorm(bf16(Kf), 0, 4), rtol=1e-14)


# =============================================================================== O2: plain top-k
def _is_valid_topk(score, kept, k, largest=False):
    """Definition: |S| = k and every kept (score, index) pair precedes every dropped pair."""
    n = len(score)
    kept = set(int(i) for i in kept)
    if len(kept) != min(k, n):
        return False
    key = [((-s if largest else s), i) for i, s in enumerate(score)]
    drop = [key[i] for i in range(n) if i not in kept]
    keep = [key[i] for i in kept]
    return not keep or not drop or max(keep) < min(drop)


@pytest.mark.parametrize("kind", ["lognormal", "ties", "equal", "signed"])
def test_select_plain_brute_force(kind):
    for n in (1, 2, 5, 9, 12):
        score = W.make_scores(5, 1, n, kind)[0].astype(np.float64)
        for k in range(0, n + 3):
            for largest in (False, True):
                got = oracle.select_plain(score, k, largest)
                assert list(got) == sorted(got), "ascending output"
                assert _is_valid_topk(score, got, k, largest)
                # uniqueness of the valid set: enumerate every subset of that size
                kk = min(k, n)
                valid = [c for c in itertools.combinations(range(n), kk) if _is_valid_topk(score, c, k, largest)]
                assert valid == [tuple(got)]


def test_select_plain_monotone_inputs():
    n, k = 17, 6
    inc = np.arange(n, dtype=np.float64)
    assert list(oracle.select_plain(inc, k)) == list(range(k))
    assert list(oracle.select_plain(-inc, k)) == list(range(n - k, n))
    assert list(oracle.select_plain(np.ones(n), k)) == list(range(k))           # ties -> lowest index
    assert list(oracle.select_plain(inc, 0)) == []
    assert list(oracle.select_plain(inc, n)) == list(range(n))
    assert list(oracle.select_plain(inc, n + 5)) == list(range(n))              # budget >= n keeps everything
    s = W.make_scores(3, 1, 40, "signed")[0].astype(np.float64)
    assert np.array_equal(oracle.select_plain(s, 11, largest=True), oracle.select_plain(-s, 11))


def test_select_smaller_norm_is_kept():
    # Stage III keeps the tokens with the SMALLEST K-norm
    s = np.array([5.0, 1.0, 4.0, 0.5, 3.0])
    assert list(oracle.select_plain(s, 2)) == [1, 3]


def test_select_nan_sorts_last():
    s = np.array([2.0, np.nan, 1.0, np.inf, 0.0])
    assert list(oracle.select_plain(s, 3)) == [0, 2, 4]
    assert list(oracle.select_plain(s, 4)) == [0, 2, 3, 4]


# =============================================================================== O4: quota (Eq. 5)
def _read_quota_examples():
    out = []
    with open(os.path.join(GOLDEN, "quota_examples.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            b, sizes, q = [p.strip() for p in line.split(";")]
            out.append((int(b), [int(x) for x in sizes.split()], [int(x) for x in q.split()]))
    return out


def test_quota_hand_examples():
    for budget, sizes, quotas in _read_quota_examples():
        n = sum(sizes)
        # cluster c occupies a contiguous run; its label is the run's first token
        label = np.concatenate([np.full(s, sum(sizes[:c]), dtype=np.int32) for c, s in enumerate(sizes)])
        score = np.arange(n, dtype=np.float64)[::-1].copy()
        keep, nc, quota = oracle.select_quota(score, label, budget)
        assert nc == len(sizes)
        got_q = [int(quota[sum(sizes[:c])]) for c in range(len(sizes))]
        assert got_q == quotas
        assert len(keep) == sum(quotas) and len(keep) + nc <= budget
        # decreasing scores -> each cluster keeps its LAST q_c members
        start = 0
        expect = []
        for s, q in zip(sizes, quotas):
            expect += list(range(start + s - q, start + s))
            start += s
        assert list(keep) == expect


def test_quota_single_cluster_equals_plain():
    s = W.make_scores(11, 1, 50, "lognormal")[0].astype(np.float64)
    label = np.full(50, 17, dtype=np.int32)
    keep, nc, _ = oracle.select_quota(s, label, 20)
    assert nc == 1
    assert np.array_equal(keep, oracle.select_plain(s, 19))        # q = (50 * 19) div 50 = 19


@pytest.mark.parametrize("kind", ["lognormal", "ties"])
def test_quota_properties_random(kind):
    n, ncl = 97, 7
    s = W.make_scores(4, 1, n, kind)[0].astype(np.float64)
    label = W.make_labels(4, 1, n, ncl)[0]
    for budget in (ncl, ncl + 1, 30, 60, n):
        keep, nc, quota = oracle.select_quota(s, label, budget)
        assert nc == len(set(label.tolist()))
        total = 0
        for c in set(label.tolist()):
            members = np.flatnonzero(label == c)
            q = (len(members) * (budget - nc)) // n                 # Eq. 5 in integers
            assert quota[c] == q
            kept_c = [i for i in keep if label[i] == c]
            assert len(kept_c) == q
            local = [int(np.flatnonzero(members == i)[0]) for i in kept_c]
            assert _is_valid_topk(s[members], local, q)             # definitional check inside the cluster
            total += q
        assert len(keep) == total <= budget - nc
        assert list(keep) == sorted(keep)
    assert oracle.select_quota(s, label, ncl - 1)[0] is None        # budget below the cluster count


# =============================================================================== O3: VIC (Alg. 2)
def _unit_rows(n, D, seed):
    rng = np.random.default_rng(seed)
    return bf16(rng.standard_normal((n, D)))


def test_similarity_basic_properties():
    f = _unit_rows(40, 64, 0)
    d2, sim = oracle.feature_distance(f, 0)
    np.testing.assert_allclose(np.diag(sim), 1.0, rtol=0, atol=1e-15)
    np.testing.assert_allclose(sim, sim.T, rtol=0, atol=1e-15)
    assert np.all(np.abs(sim) <= 1 + 1e-15)
    np.testing.assert_allclose(d2, np.maximum(0, 2 - 2 * sim), atol=1e-15)
    # cosine distance is the Euclidean distance between the L2-normalised rows (numpy, independent route)
    x = W.bf16_bits_to_f32(f).astype(np.float64)
    xn = x / np.linalg.norm(x, axis=1, keepdims=True)
    ref = ((xn[:, None, :] - xn[None, :, :]) ** 2).sum(-1)
    np.testing.assert_allclose(d2, ref, atol=1e-13)
    # euclid metric: plain squared distance; "sim" is then the raw Gram matrix
    d2e, g = oracle.feature_distance(f, 1)
    np.testing.assert_allclose(d2e, ((x[:, None, :] - x[None, :, :]) ** 2).sum(-1), rtol=1e-12, atol=1e-10)
    np.testing.assert_allclose(g, x @ x.T, rtol=1e-12, atol=1e-12)
    # a row block equals the same rows of the full matrix
    d2r, simr = oracle.feature_distance(f, 0, rows=(7, 19))
    assert np.array_equal(d2r, d2[7:19]) and np.array_equal(simr, sim[7:19])


def test_similarity_hand_values():
    # f0 = (1,0), f1 = (1,1), f2 = (0,2), f3 = (-1,0):  cos(0,1) = 1/sqrt2, cos(0,2) = 0, cos(0,3) = -1
    f = bf16([[1, 0], [1, 1], [0, 2], [-1, 0]])
    d2, sim = oracle.feature_distance(f, 0)
    r = 1 / math.sqrt(2)
    np.testing.assert_allclose(sim[0], [1, r, 0, -1], atol=1e-15)
    np.testing.assert_allclose(d2[0], [0, 2 - 2 * r, 2, 4], atol=1e-15)
    np.testing.assert_allclose(sim[1, 2], r, atol=1e-15)
    # Eq. 2 by hand for token 0 with d_c = 0.5
    rho = oracle.vic_density(d2, 0.5)
    expect0 = math.exp(-(2 - 2 * r) / 0.25) + math.exp(-2 / 0.25) + math.exp(-4 / 0.25)
    assert abs(rho[0] - expect0) < 1e-15
    # zero-norm feature: similarity 0 against everything, d2 = 2
    d2z, simz = oracle.feature_distance(bf16([[0, 0], [1, 0]]), 0)
    assert simz[0, 1] == 0 and d2z[0, 1] == 2


def test_density_closed_forms():
    n, dc = 16, 0.7
    eye = bf16(np.eye(n) * 3.0)                         # orthogonal rows: s = 0, d^2 = 2
    d2, _ = oracle.feature_distance(eye, 0)
    assert np.all(d2[~np.eye(n, dtype=bool)] == 2.0)
    rho = oracle.vic_density(d2, dc)
    np.testing.assert_allclose(rho, (n - 1) * math.exp(-2 / dc ** 2), rtol=1e-14)
    same = bf16(np.tile(np.array([[1.0, -2.0, 0.5]]), (n, 1)))   # n identical tokens: every term is exp(0)
    d2s, _ = oracle.feature_distance(same, 0)
    np.testing.assert_allclose(d2s, 0, atol=1e-15)
    np.testing.assert_allclose(oracle.vic_density(d2s, dc), n - 1, rtol=1e-14)


def test_identical_tokens_single_cluster():
    n = 9
    f = bf16(np.tile(np.array([[1.0, 2.0, 3.0, 4.0]]), (n, 1)))
    r = oracle.vic(f, None, 0, 0.5, -1.0, 1)
    assert r["is_center"].tolist() == [1] + [0] * (n - 1)   # equal densities: the lowest index is densest
    assert np.all(r["label"] == 0)
    assert r["parent"].tolist() == [-1] + [0] * (n - 1)     # ties in distance -> lowest index
    assert math.isinf(r["delta2"][0]) and np.all(r["delta2"][1:] < 1e-15)


def test_exact_duplicates_share_a_cluster():
    w = W.workload("tiny")
    f = W.make_features(w)[0].copy()
    p = W.make_positions(w)[0]
    f[31] = f[30]                                        # neighbours on the 24-grid, inside tau
    f[101] = f[100]
    r = oracle.vic(f, p, 0, w.d_c, w.tau, w.n_centers)
    assert r["sim"][30, 31] == pytest.approx(1.0, abs=1e-15) and r["d2"][30, 31] < 1e-15
    assert r["label"][30] == r["label"][31] and r["label"][100] == r["label"][101]


def test_two_separated_groups():
    rng = np.random.default_rng(5)
    a = np.array([1.0, 0, 0, 0]) + 0.02 * rng.standard_normal((6, 4))
    b = np.array([0, 0, 1.0, 0]) + 0.02 * rng.standard_normal((8, 4))
    f = bf16(np.concatenate([a, b]))
    r = oracle.vic(f, None, 0, 0.5, -1.0, 2)
    la, lb = set(r["label"][:6].tolist()), set(r["label"][6:].tolist())
    assert len(la) == 1 and len(lb) == 1 and la != lb
    assert list(la)[0] < 6 <= list(lb)[0]                # each label is a token of its own group


def _density_peaks_bruteforce(x, dc, n_centers):
    """Independent restatement (pure Python) of density-peaks clustering with a Gaussian kernel."""
    n = len(x)
    xn = [v / np.linalg.norm(v) for v in x]
    d = [[float(np.linalg.norm(xn[i] - xn[j])) for j in range(n)] for i in range(n)]
    rho = [sum(math.exp(-(d[i][j] / dc) ** 2) for j in range(n) if j != i) for i in range(n)]
    parent, delta = [], []
    for i in range(n):
        cand = [(d[i][j], j) for j in range(n) if j != i and (rho[j] > rho[i] or (rho[j] == rho[i] and j < i))]
        if cand:
            dd, j = min(cand)
            parent.append(j), delta.append(dd)
        else:
            parent.append(-1), delta.append(math.inf)
    gamma = [rho[i] * delta[i] if parent[i] >= 0 else math.inf for i in range(n)]
    order = sorted(range(n), key=lambda i: (-gamma[i], -rho[i], i))
    centres = set(order[:n_centers])
    label = [-1] * n
    for i in sorted(range(n), key=lambda i: (-rho[i], i)):
        if i in centres:
            label[i] = i
        elif parent[i] >= 0:
            label[i] = label[parent[i]]
        else:
            label[i] = min((d[i][c], c) for c in centres)[1]
    return rho, delta, parent, sorted(centres), label


@pytest.mark.parametrize("seed,n,nc", [(0, 24, 3), (1, 48, 5), (2, 64, 4)])
def test_vic_without_spatial_mask_is_density_peaks(seed, n, nc):
    rng = np.random.default_rng(seed)
    centres = rng.standard_normal((nc, 12))
    x = centres[rng.integers(0, nc, n)] + 0.3 * rng.standard_normal((n, 12))
    fb = bf16(x)
    xf = W.bf16_bits_to_f32(fb).astype(np.float64)
    rho, delta, parent, cs, label = _density_peaks_bruteforce(xf, 0.5, nc)
    pos = rng.random((n, 2)).astype(np.float32)
    for kwargs in (dict(pos=None, tau=-1.0), dict(pos=pos, tau=1e9)):        # tau = infinity: mask is vacuous
        r = oracle.vic(fb, kwargs["pos"], 0, 0.5, kwargs["tau"], nc)
        np.testing.assert_allclose(r["rho"], rho, rtol=1e-12)
        assert r["parent"].tolist() == parent
        fin = np.isfinite(r["delta2"])
        np.testing.assert_allclose(np.sqrt(r["delta2"][fin]), np.array(delta)[fin], atol=1e-7)
        assert np.flatnonzero(r["is_center"]).tolist() == cs
        assert r["label"].tolist() == label


def test_spatial_mask_hand_example():
    # unit vectors at angles 0, 0.1, 0.2, 0.9 rad: chord distance ~ angle, so with d_c = 0.5 the
    # densities fall in the order 1 > 2 > 0 > 3 (token 1 sits in the middle of the tight triple)
    ang = np.array([0.0, 0.1, 0.2, 0.9])
    f = bf16(np.stack([np.cos(ang), np.sin(ang)], 1))
    d2, _ = oracle.feature_distance(f, 0)
    rho = oracle.vic_density(d2, 0.5)
    assert sorted(range(4), key=lambda i: -rho[i]) == [1, 2, 0, 3]
    # no mask: everybody points at the nearest denser token in feature space
    delta2, parent, _ = oracle.vic_parents(d2, None, rho, -1.0)
    assert parent.tolist() == [1, -1, 1, 2] and math.isinf(delta2[1])
    assert delta2[3] == d2[3, 2] and delta2[0] == d2[0, 1]
    # tokens laid out on a line at x = 0, 0.1, 0.9, 1.0
    pos = np.array([[0.0, 0.0], [0.1, 0.0], [0.9, 0.0], [1.0, 0.0]], dtype=np.float32)
    # tau = 0.15: 3 sees only 2; 0 sees only 1; 2 sees only 3 (less dense) and 1 only 0 (less dense)
    delta2, parent, _ = oracle.vic_parents(d2, pos, rho, 0.15)
    assert parent.tolist() == [1, -1, -1, 2] and math.isinf(delta2[2])
    # tau = 0.05: nobody sees anybody
    delta2, parent, _ = oracle.vic_parents(d2, pos, rho, 0.05)
    assert parent.tolist() == [-1] * 4 and np.all(np.isinf(delta2))
    # the mask redirects token 0: its nearest denser token (1) is far away in the image, token 2 is close
    pos = np.array([[0.0, 0.0], [1.0, 0.0], [0.1, 0.0], [0.5, 0.5]], dtype=np.float32)
    delta2, parent, _ = oracle.vic_parents(d2, pos, rho, 0.5)
    assert parent[0] == 2 and delta2[0] == d2[0, 2] and delta2[0] > d2[0, 1]
    # a pair exactly tau apart is admitted ("<= tau"), just below it is not
    pos = np.array([[0.0, 0.0], [0.5, 0.0], [0.0, 0.75], [0.75, 0.75]], dtype=np.float32)
    assert oracle.vic_parents(d2, pos, rho, 0.5)[1][0] == 1
    assert oracle.vic_parents(d2, pos, rho, 0.4999)[1][0] == -1


# The robustness report of oracle.vic_parents decides which tokens a lower-precision implementation may
# legitimately disagree on, so its band must be neither too narrow nor too wide.  Hand-built cases: the answer is
# known by construction on each side of every tolerance.
def _frag(d2, pos, rho, tau, **tols):
    _, parent, frag = oracle.vic_parents(np.asarray(d2, dtype=np.float64), pos, np.asarray(rho, dtype=np.float64),
                                         tau, want_fragile=True, **tols)
    return parent.tolist(), frag.astype(bool).tolist()


def _sym(n, entries, fill=9.0):
    d2 = np.full((n, n), fill)
    np.fill_diagonal(d2, 0.0)
    for (i, j), v in entries.items():
        d2[i, j] = d2[j, i] = v
    return d2


@pytest.mark.parametrize("factor,expect", [(0.5, True), (2.0, False)])
def test_fragile_report_distance_band(factor, expect):
    # token 0 has two denser candidates: 1 at d2 = 1 (the parent) and 2 at d2 = 1 + factor * band, where
    # band = tol_abs + tol_rel * 1: half a band away the runner-up could win, two bands away it could not
    tol_abs, tol_rel = 3e-6, 1e-5
    band = tol_abs + tol_rel * 1.0
    d2 = _sym(3, {(0, 1): 1.0, (0, 2): 1.0 + factor * band, (1, 2): 4.0})
    parent, frag = _frag(d2, None, [1.0, 2.0, 3.0], -1.0, tol_d2_abs=tol_abs, tol_d2_rel=tol_rel)
    assert parent == [1, 2, -1]
    assert frag == [expect, False, False]
    # the absolute and the relative part each count on their own
    for kw in (dict(tol_d2_abs=band), dict(tol_d2_rel=band)):
        assert _frag(d2, None, [1.0, 2.0, 3.0], -1.0, **kw)[1][0] is expect


@pytest.mark.parametrize("factor,expect", [(0.5, True), (2.0, False)])
def test_fragile_report_density_band(factor, expect):
    tol = 1e-4
    # (a) a closer token whose density lies just BELOW token 0's: not a candidate, but it could become one
    rho = [1.0, 2.0, 1.0 - factor * tol]
    d2 = _sym(3, {(0, 1): 1.0, (0, 2): 0.25, (1, 2): 4.0})
    parent, frag = _frag(d2, None, rho, -1.0, tol_rho=tol)
    assert parent[0] == 1 and frag[0] is expect
    # (b) the parent's own density lies just ABOVE token 0's: it could stop being a candidate
    rho = [1.0, 1.0 + factor * tol, 0.5]
    parent, frag = _frag(_sym(3, {(0, 1): 1.0, (0, 2): 0.25, (1, 2): 4.0}), None, rho, -1.0, tol_rho=tol)
    assert parent[0] == 1 and frag[0] is expect
    # (c) an orphan (densest token) with a near-equal neighbour could gain a parent
    rho = [1.0, 1.0 - factor * tol, 0.5]
    parent, frag = _frag(_sym(3, {(0, 1): 1.0}), None, rho, -1.0, tol_rho=tol)
    assert parent[0] == -1 and frag[0] is expect
    # a farther token cannot matter however close its density is
    rho = [1.0, 2.0, 1.0 - 0.5 * tol]
    assert _frag(_sym(3, {(0, 1): 1.0, (0, 2): 1.5, (1, 2): 4.0}), None, rho, -1.0, tol_rho=tol)[1][0] is False


@pytest.mark.parametrize("factor,expect", [(0.5, True), (2.0, False)])
def test_fragile_report_spatial_band(factor, expect):
    tau, tol = 0.5, 1e-3                                   # positions on the x axis: distances exact in fp32 -> fp64
    x = lambda v: np.array([[0.0, 0.0], [np.float32(v), 0.0], [0.25, 0.0]], dtype=np.float32)
    rho = [1.0, 2.0, 3.0]
    # (a) a closer, denser token just OUTSIDE the radius: excluded, but it could slip inside
    d2 = _sym(3, {(0, 1): 0.25, (0, 2): 1.0, (1, 2): 4.0})
    parent, frag = _frag(d2, x(tau * (1 + factor * tol)), rho, tau, tol_sp=tol)
    assert parent[0] == 2 and frag[0] is expect
    # (b) the parent itself just INSIDE the radius: it could slip outside
    d2 = _sym(3, {(0, 1): 0.25, (0, 2): 1.0, (1, 2): 4.0})
    parent, frag = _frag(d2, x(tau * (1 - factor * tol)), rho, tau, tol_sp=tol)
    assert parent[0] == 1 and frag[0] is expect


def test_fragile_report_without_tolerances_flags_exact_ties_only():
    rng = np.random.default_rng(5)
    n = 80
    a = rng.random((n, n)) + 0.1
    d2 = (a + a.T) / 2
    np.fill_diagonal(d2, 0.0)
    rho = rng.random(n) + 1.0
    pos = rng.random((n, 2)).astype(np.float32)
    for kw in (dict(pos=None, tau=-1.0), dict(pos=pos, tau=0.45)):
        parent, frag = _frag(d2, kw["pos"], rho, kw["tau"])
        assert not any(frag)                               # continuous random values: no ties, nothing fragile
    # plant (1) an exact tie in distance between the parent of token t and another denser token, and
    #       (2) an exact tie in density between a token u and a closer token
    parent, _ = _frag(d2, None, rho, -1.0)
    order = np.argsort(rho)
    t = int(order[10])                                     # a token with many denser ones
    denser = [int(j) for j in order[11:] if j != parent[t]]
    other = denser[0]
    d2b = d2.copy()
    for j in (other, parent[t]):                           # both at the same distance, closer than everything else
        d2b[t, j] = d2b[j, t] = 2e-3
    u = int(order[30])
    v = int(order[5])                                      # strictly less dense than u ...
    rho_b = rho.copy()
    rho_b[v] = rho_b[u]                                    # ... now exactly as dense
    d2b[u, v] = d2b[v, u] = 1e-3                           # and closer than anything else
    parent_b, frag_b = _frag(d2b, None, rho_b, -1.0)
    flagged = set(np.flatnonzero(frag_b).tolist())
    assert t in flagged and u in flagged and v in flagged
    # every flagged token owes it to one of the two planted ties
    for i in flagged:
        best = d2b[i, parent_b[i]] if parent_b[i] >= 0 else np.inf
        ties_d = [j for j in range(n) if j not in (i, parent_b[i]) and rho_b[j] >= rho_b[i] and d2b[i, j] == best]
        ties_r = [j for j in range(n) if j != i and rho_b[j] == rho_b[i] and d2b[i, j] <= best]
        assert ties_d or ties_r, i


def test_all_orphans_fall_back_to_nearest_centre():
    w = W.workload("tiny")
    f = W.make_features(w)[0][:60]
    p = W.make_positions(w)[0][:60]
    r = oracle.vic(f, p, 0, w.d_c, 0.0, 5)               # tau = 0, distinct positions: no admissible neighbour
    assert np.all(r["parent"] == -1) and np.all(np.isinf(r["delta2"]))
    cs = np.flatnonzero(r["is_center"])
    assert cs.tolist() == sorted(np.argsort(-r["rho"], kind="stable")[:5].tolist())   # orphans rank by density
    for i in range(60):
        if i in cs:
            assert r["label"][i] == i
        else:
            assert r["label"][i] == cs[np.argmin(r["d2"][i, cs])]


@pytest.mark.parametrize("name", ["tiny", "c0"])
def test_vic_invariants(name):
    w = W.workload(name)
    f = W.make_features(w)[0]
    p = W.make_positions(w)[0]
    r = oracle.vic(f, p, 0, w.d_c, w.tau, w.n_centers)
    n = f.shape[0]
    rho, parent, label = r["rho"], r["parent"], r["label"]
    cs = set(np.flatnonzero(r["is_center"]).tolist())
    assert len(cs) == w.n_centers == r["n_clusters"]
    assert set(label.tolist()) == cs                     # every label is a centre, every centre is used
    for i in range(n):
        j = parent[i]
        if j >= 0:
            assert rho[j] > rho[i] or (rho[j] == rho[i] and j < i)          # chains climb in density: no cycles
            assert np.hypot(*(p[i].astype(np.float64) - p[j].astype(np.float64))) <= w.tau
            assert r["delta2"][i] == r["d2"][i, j]
        if i in cs:
            assert label[i] == i
        elif j >= 0:
            assert label[i] == label[j]
    # permuting feature dimensions or scaling by a power of two changes nothing discrete
    perm = np.random.default_rng(0).permutation(f.shape[1])
    r2 = oracle.vic(f[:, perm], p, 0, w.d_c, w.tau, w.n_centers)
    np.testing.assert_allclose(r2["rho"], rho, rtol=1e-12)
    r3 = oracle.vic(bf16(W.bf16_bits_to_f32(f) * 4.0), p, 0, w.d_c, w.tau, w.n_centers)
    assert np.array_equal(r3["rho"], rho) and np.array_equal(r3["label"], label)
    # near-duplicate tokens (sigma 0.01 copies) end up with their source
    d2 = r["d2"] + np.eye(n) * 9
    close = np.argwhere(d2 < 1e-3)
    assert len(close) > 0
    same = sum(label[a] == label[b] for a, b in close)
    assert same >= 0.9 * len(close)


def test_num_centers_ceiling():
    assert oracle.vic_num_centers(576, 0.05) == 29       # ceil(28.8)
    assert oracle.vic_num_centers(100, 0.05) == 5        # exact product: no spurious +1
    assert oracle.vic_num_centers(10, 0.0) == 0
    assert oracle.vic_num_centers(10, 2.0) == 10


# =============================================================================== O5: compaction
def _toy_sequence(N=23, H=3, d=8, Dh=16, seed=0):
    rng = np.random.default_rng(seed)
    return (rng.integers(0, 65536, (N, Dh)).astype(np.uint16), rng.integers(0, 65536, (H, N, d)).astype(np.uint16),
            rng.integers(0, 65536, (H, N, d)).astype(np.uint16))


def test_compact_identity_and_none():
    hid, K, V = _toy_sequence()
    N = hid.shape[0]
    vs, vl = 4, 12
    r = oracle.compact(hid, K, V, N, vs, vl, np.arange(vl), N)
    assert r["out_len"] == N and np.array_equal(r["hidden"], hid) and np.array_equal(r["K"], K) and np.array_equal(r["V"], V)
    assert r["kept_pos"].tolist() == list(range(N))
    r = oracle.compact(hid, K, V, N, vs, vl, np.zeros(0, np.int32), N)
    text = list(range(vs)) + list(range(vs + vl, N))
    assert r["out_len"] == N - vl and r["kept_pos"][: N - vl].tolist() == text
    assert np.array_equal(r["hidden"][: N - vl], hid[text]) and np.array_equal(r["K"][:, : N - vl], K[:, text])


def test_compact_rows_and_order():
    hid, K, V = _toy_sequence(seed=1)
    N, vs, vl = hid.shape[0], 5, 10
    keep = np.array([1, 2, 7, 9], dtype=np.int32)
    r = oracle.compact(hid, K, V, N, vs, vl, keep, N)
    src = list(range(vs)) + [vs + k for k in keep] + list(range(vs + vl, N))
    L = r["out_len"]
    assert L == len(src) and r["kept_pos"][:L].tolist() == src
    assert np.all(np.diff(r["kept_pos"][:L]) > 0)
    assert np.array_equal(r["hidden"][:L], hid[src]) and np.array_equal(r["V"][:, :L], V[:, src])
    assert np.all(r["hidden"][L:] == 0)
    # a shorter sequence inside a longer buffer: rows past seq_len are ignored
    r2 = oracle.compact(hid, K, V, N - 3, vs, vl, keep, N)
    assert r2["out_len"] == L - 3 and np.array_equal(r2["K"][:, : L - 3], K[:, src[:-3]])


def test_compact_composes():
    hid, K, V = _toy_sequence(N=40, seed=2)
    N, vs, vl = 40, 6, 30
    a = np.array(sorted(np.random.default_rng(0).permutation(vl)[:17]), dtype=np.int32)
    b = np.array(sorted(np.random.default_rng(1).permutation(17)[:6]), dtype=np.int32)
    r1 = oracle.compact(hid, K, V, N, vs, vl, a, N)
    L1 = r1["out_len"]
    r2 = oracle.compact(r1["hidden"], r1["K"], r1["V"], L1, vs, 17, b, N)
    rc = oracle.compact(hid, K, V, N, vs, vl, a[b], N)
    L = rc["out_len"]
    assert r2["out_len"] == L
    assert np.array_equal(r2["hidden"][:L], rc["hidden"][:L]) and np.array_equal(r2["K"][:, :L], rc["K"][:, :L])
    assert np.array_equal(r1["kept_pos"][:L1][r2["kept_pos"][:L]], rc["kept_pos"][:L])


# =============================================================================== schedule (Alg. 1, Eq. 10)
def test_retention_table_counts_and_compression():
    rows = [list(map(float, l.split())) for l in open(os.path.join(GOLDEN, "retention_ratios.txt"))
            if l.strip() and not l.startswith("#")]
    m = 576
    nominal = {66.7: 192, 77.8: 128, 88.9: 64, 94.4: 32}
    counts = {}
    for rate, p1, p2, p3 in rows:
        c = tuple(oracle.stage_count(m, p) for p in (p1, p2, p3))
        counts[rate] = c
        assert c[0] > c[1] > c[2] > 0
        # the printed overall rate is 1 - nominal/576; Eq. 10 averaged over the 32 layers (l_s = 2, l_d = 22)
        # reproduces it to within a few percent of the token count
        assert abs((1 - nominal[rate] / m) * 100 - rate) < 0.06
        cr = oracle.cr_int(p1, p2, p3, 2, 22, 32)
        assert abs(cr - rate / 100) < 0.02
        assert abs(cr - (1 - (p1 * 1 + p2 * 20 + p3 * 11) / 32)) < 1e-15
    assert counts[66.7] == (288, 253, 50) and counts[88.9] == (172, 77, 15)
    assert counts[77.8] == (230, 165, 33) and counts[94.4] == (144, 33, 6)


def test_chain_kept_count_equals_budget():
    # Stage III chain on the tiny workload: kept count == min(budget, n) at every step
    w = W.workload("tiny")
    n = w.Nv
    for step, k in enumerate(w.budgets):
        K, _ = W.make_kv(w, step, n)
        s = oracle.knorm(K, w.vis_start, n)
        for b in range(w.B):
            keep = oracle.select_plain(s[b], k)
            assert len(keep) == min(k, n)
        n = min(k, n)


# ======================================================================================= Eq. 6: cluster merge
def test_merge_hand_example():
    # four tokens, Dh = 2, labels {0,0,2,2}, token 0 kept: cluster 0 averages token 1 alone, cluster 2 averages 2 and 3
    hid = W.f32_to_bf16_bits(np.array([[9, 9], [1, 2], [3, 5], [4, 6], [5, 7]], dtype=np.float32))   # row 0 is text
    merged, mlab, mcnt = oracle.merge_clusters(hid, 1, np.array([0, 0, 2, 2]), np.array([1, 0, 0, 0]))
    assert mlab.tolist() == [0, 2] and mcnt.tolist() == [1, 2]
    assert np.array_equal(merged, np.array([[3.0, 5.0], [4.5, 6.5]]))
    # every token of a cluster kept -> no merged row for it
    merged, mlab, mcnt = oracle.merge_clusters(hid, 1, np.array([0, 0, 2, 2]), np.array([1, 1, 0, 1]))
    assert mlab.tolist() == [2] and mcnt.tolist() == [1] and np.array_equal(merged, np.array([[4.0, 6.0]]))


def test_merge_conservation_and_library_mean():
    rng = np.random.default_rng(5)
    n, Dh, vs = 97, 24, 3
    hid = W.f32_to_bf16_bits(rng.standard_normal((vs + n + 2, Dh)).astype(np.float32))
    x = W.bf16_bits_to_f32(hid).astype(np.float64)[vs:vs + n]
    label = W.make_labels(3, 1, n, 7)[0]
    keep = (rng.random(n) < 0.3).astype(np.uint8)
    merged, mlab, mcnt = oracle.merge_clusters(hid, vs, label, keep)
    # counts: every non-elite token is averaged exactly once
    assert mcnt.sum() == n - keep.sum() and np.all(np.diff(mlab) > 0)
    # conservation: sum_c count_c * merged_c + sum of elite rows == sum of all rows
    assert np.allclose((merged * mcnt[:, None]).sum(0) + x[keep == 1].sum(0), x.sum(0), rtol=0, atol=1e-10)
    # each row against numpy's mean over the members
    for r, lab in enumerate(mlab):
        members = (label == lab) & (keep == 0)
        assert np.allclose(merged[r], x[members].mean(0), rtol=0, atol=1e-13)
    # a single cluster with nothing kept is the plain column mean; constant rows average to the constant
    merged, _, mcnt = oracle.merge_clusters(hid, vs, np.zeros(n, np.int32), np.zeros(n, np.uint8))
    assert mcnt.tolist() == [n] and np.allclose(merged[0], x.mean(0), atol=1e-13)
    const = W.f32_to_bf16_bits(np.full((n, Dh), 1.5, dtype=np.float32))
    merged, _, _ = oracle.merge_clusters(const, 0, label, keep)
    assert np.all(merged == 1.5)


# ======================================================================================= Eq. 1: [CLS] saliency
def test_cls_saliency_closed_forms():
    H, M, d = 4, 33, 16
    rng = np.random.default_rng(2)
    q = W.f32_to_bf16_bits(rng.standard_normal((H, d)).astype(np.float32))
    # identical keys: every attention row is uniform, S_i = H / M
    K = np.tile(W.f32_to_bf16_bits(rng.standard_normal((H, 1, d)).astype(np.float32)), (1, M, 1))
    S, c = oracle.cls_saliency(q, K, 0.25)
    assert np.allclose(S, H / M, atol=1e-14) and abs(c - H / M) < 1e-14
    # each head's row sums to one: [CLS] share + visual shares == H
    K = W.f32_to_bf16_bits(rng.standard_normal((H, M, d)).astype(np.float32))
    S, c = oracle.cls_saliency(q, K, 0.25)
    assert abs(S.sum() + c - H) < 1e-12 and np.all(S > 0)
    # against a library softmax on the same logits
    from scipy.special import softmax
    qf, Kf = W.bf16_bits_to_f32(q).astype(np.float64), W.bf16_bits_to_f32(K).astype(np.float64)
    ref = softmax(0.25 * np.einsum("hd,hmd->hm", qf, Kf), axis=1).sum(0)
    assert np.allclose(S, ref[1:], rtol=1e-12, atol=0)
    # shifting every key by one vector adds the same constant to all logits of a head: S unchanged
    shift = W.bf16_bits_to_f32(W.f32_to_bf16_bits(np.full((1, 1, d), 0.5, dtype=np.float32)))
    K2 = W.f32_to_bf16_bits((W.bf16_bits_to_f32(K) * 0.5).astype(np.float32))       # exact halving keeps bf16 exact
    K3 = W.f32_to_bf16_bits((W.bf16_bits_to_f32(K2) + shift).astype(np.float32))
    exact = np.array_equal(W.bf16_bits_to_f32(K3), W.bf16_bits_to_f32(K2) + shift)
    S2, _ = oracle.cls_saliency(q, K2, 0.25)
    S3, _ = oracle.cls_saliency(q, K3, 0.25)
    if exact:
        assert np.allclose(S2, S3, rtol=1e-10)
    # one key aligned with the query and a large scale: that token takes (almost) all the attention of every head
    K = np.zeros((H, M, d), dtype=np.float32)
    K[:, 7] = W.bf16_bits_to_f32(q)
    S, c = oracle.cls_saliency(q, W.f32_to_bf16_bits(K), 50.0)
    assert abs(S[6] - H) < 1e-6 and S[6] == S.max()


# ======================================================================================= Eq. 7-9: cost model
def test_cost_model_closed_forms():
    assert oracle.flops_layer(1, 1) == 20.0
    assert oracle.flops_layer(3, 2) == 4 * 9 * 2 + 16 * 3 * 4
    # Eq. 8 boundaries with l_s = 2, l_d = 22
    m, p = 576.0, (0.5, 0.4394, 0.0879)
    assert oracle.visual_tokens_at_layer(1, m, *p) == 0.5 * m
    assert oracle.visual_tokens_at_layer(2, m, *p) == 0.4394 * m == oracle.visual_tokens_at_layer(21, m, *p)
    assert oracle.visual_tokens_at_layer(22, m, *p) == 0.0879 * m == oracle.visual_tokens_at_layer(32, m, *p)
    # Eq. 9 is the sum of Eq. 7 over the layers with the token count of Eq. 8
    tot = sum(oracle.flops_layer(oracle.visual_tokens_at_layer(l, m, *p) + 64, 4096) for l in range(1, 33))
    assert abs(oracle.flops_vitcop(m, 64, 4096, *p) - tot) <= 1e-9 * tot
    # no pruning: n layers at full length; Eq. 10 is then zero
    assert oracle.flops_vitcop(m, 64, 4096, 1, 1, 1) == 32 * oracle.flops_layer(m + 64, 4096)
    assert oracle.cr_int(1, 1, 1) == 0.0
    # Eq. 10 equals one minus the layer average of Eq. 8 over m
    avg = sum(oracle.visual_tokens_at_layer(l, m, *p) for l in range(1, 33)) / (32 * m)
    assert abs(oracle.cr_int(*p) - (1 - avg)) < 1e-15


# =============================================================================== O9: K projection + K-norm
def test_kproj_identity_weights_reduce_to_knorm():
    # W = I (H * d == Dh): K is the hidden row cut into heads, so the score is Eq. 4 of that tensor
    rng = np.random.default_rng(7)
    N, H, d = 9, 4, 8
    hid = bf16(rng.standard_normal((N, H * d)))
    W_id = bf16(np.eye(H * d))
    K64, Kb, score = oracle.kproj_knorm(hid, W_id, H, d)
    as_K = np.ascontiguousarray(hid.reshape(N, H, d).transpose(1, 0, 2))          # [H, N, d]
    assert np.array_equal(Kb, as_K)
    assert np.array_equal(K64, W.bf16_bits_to_f32(as_K).astype(np.float64))
    assert np.array_equal(score, oracle.knorm(as_K[None], 0, N)[0])


def test_kproj_one_hot_weights_pick_hidden_elements():
    rng = np.random.default_rng(8)
    N, Dh, H, d = 5, 24, 2, 4
    hid = bf16(rng.standard_normal((N, Dh)))
    pick = rng.permutation(Dh)[: H * d]
    Wm = np.zeros((H * d, Dh), dtype=np.float32)
    Wm[np.arange(H * d), pick] = -2.0                       # scaling by a power of two is exact
    K64, Kb, score = oracle.kproj_knorm(hid, bf16(Wm), H, d)
    want = -2.0 * W.bf16_bits_to_f32(hid).astype(np.float64)[:, pick].reshape(N, H, d).transpose(1, 0, 2)
    assert np.array_equal(K64, want)
    np.testing.assert_allclose(score, np.sqrt((want ** 2).sum((0, 2))), rtol=1e-14)


def test_kproj_matches_a_matmul_and_rounds_to_nearest_even():
    rng = np.random.default_rng(9)
    N, Dh, H, d = 7, 40, 3, 8
    hid, Wk = bf16(rng.standard_normal((N, Dh))), bf16(rng.standard_normal((H * d, Dh)) * 0.2)
    K64, Kb, score = oracle.kproj_knorm(hid, Wk, H, d)
    ref = W.bf16_bits_to_f32(hid).astype(np.float64) @ W.bf16_bits_to_f32(Wk).astype(np.float64).T      # [N, H*d]
    np.testing.assert_allclose(K64, ref.reshape(N, H, d).transpose(1, 0, 2), rtol=1e-13, atol=1e-13)
    assert np.array_equal(Kb, W.f32_to_bf16_bits(K64.astype(np.float32)))                               # the repo's own rounding
    Kr = W.bf16_bits_to_f32(Kb).astype(np.float64)
    np.testing.assert_allclose(score, np.sqrt((Kr ** 2).sum((0, 2))), rtol=1e-14)
    assert np.array_equal(score, oracle.knorm(Kb[None], 0, N)[0])                                       # Eq. 4 of the rounded K


def test_kproj_rotary_embedding_quarter_turn_and_norm_invariance():
    rng = np.random.default_rng(10)
    N, Dh, H, d = 6, 16, 2, 8
    hid, Wk = bf16(rng.standard_normal((N, Dh))), bf16(rng.standard_normal((H * d, Dh)))
    plain, _, _ = oracle.kproj_knorm(hid, Wk, H, d)
    # a quarter turn at every position: (a, b) -> (-b, a) for the pairs (e, e + d/2)
    cos, sin = np.zeros((N, d // 2)), np.ones((N, d // 2))
    rot, _, _ = oracle.kproj_knorm(hid, Wk, H, d, cos, sin)
    assert np.array_equal(rot[..., : d // 2], -plain[..., d // 2:]) and np.array_equal(rot[..., d // 2:], plain[..., : d // 2])
    # any angles: the norm before rounding is unchanged; positions select the table row
    ang = rng.random((50, d // 2)) * 6.0
    position = rng.integers(0, 50, size=N).astype(np.int32)
    rot, _, _ = oracle.kproj_knorm(hid, Wk, H, d, np.cos(ang), np.sin(ang), position)
    np.testing.assert_allclose((rot ** 2).sum((0, 2)), (plain ** 2).sum((0, 2)), rtol=1e-12)
    a, b = plain[1, 3, 2], plain[1, 3, 2 + d // 2]
    c, s_ = np.cos(ang[position[3], 2]), np.sin(ang[position[3], 2])
    assert abs(rot[1, 3, 2] - (a * c - b * s_)) < 1e-12 and abs(rot[1, 3, 2 + d // 2] - (b * c + a * s_)) < 1e-12
