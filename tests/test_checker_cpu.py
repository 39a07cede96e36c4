"""The comparison rules the GPU parity tests apply (tests/gpu_helpers.py), exercised on the CPU: fed with the
oracle's own results rounded to fp32 they must pass, and a mistake planted in those results must fail them.
No CUDA call is made."""
import numpy as np
import pytest

import oracle
from paper_2601_17818_b200 import workloads as W

from gpu_helpers import KNORM_RTOL, check_vic_sample, oracle_quota_band_check


def _oracle_as_gpu(name="tiny", b=0):
    w = W.workload(name)
    f, p = W.make_features(w)[b], W.make_positions(w)[b]
    o = oracle.vic(f, p, 0, w.d_c, w.tau, w.n_centers)
    g = dict(rho=o["rho"].astype(np.float32), delta2=o["delta2"].astype(np.float32), parent=o["parent"].copy(),
             label=o["label"].copy())
    return w, f, p, o, g


def _check(w, f, p, g, **kw):
    rep = []
    check_vic_sample(f, p, 0, w.d_c, w.tau, w.n_centers, g["rho"], g["delta2"], g["parent"], g["label"], rep, **kw)
    return rep[0]


@pytest.mark.parametrize("name", ["tiny", "c0"])
def test_checker_accepts_the_oracle_itself(name):
    w, f, p, o, g = _oracle_as_gpu(name)
    st = _check(w, f, p, g)
    assert st["parent_mismatch"] == 0 and st["centre_diff"] == 0 and st["label_mismatch"] == 0
    assert st["label_uncompared"] <= 2                       # only surplus orphans with a near-tie can be left out


def test_checker_rejects_planted_mistakes():
    w, f, p, o, g = _oracle_as_gpu("tiny")
    n = len(g["label"])
    cs = np.flatnonzero(o["is_center"])
    # a wrong label on a token with a robust path
    bad = {k: v.copy() for k, v in g.items()}
    i = int(np.flatnonzero(~o["is_center"].astype(bool) & (o["parent"] >= 0))[0])
    bad["label"][i] = cs[0] if g["label"][i] != cs[0] else cs[1]
    with pytest.raises(AssertionError):
        _check(w, f, p, bad)
    # a density off by 1e-4 relative
    bad = {k: v.copy() for k, v in g.items()}
    bad["rho"][3] *= np.float32(1 + 1e-4)
    with pytest.raises(AssertionError):
        _check(w, f, p, bad)
    # a non-fragile token pointing at the wrong parent
    tol = dict(tol_rho=1e-5, tol_d2_abs=4e-6, tol_d2_rel=1e-5, tol_sp=1e-6)
    frag = oracle.vic(f, p, 0, w.d_c, w.tau, w.n_centers, tols=tol)["fragile"].astype(bool)
    bad = {k: v.copy() for k, v in g.items()}
    i = int(np.flatnonzero(~frag & (o["parent"] >= 0))[0])
    bad["parent"][i] = (o["parent"][i] + 1) % n
    with pytest.raises(AssertionError):
        _check(w, f, p, bad)
    # the lowest-gamma token promoted to a centre in place of a real one
    bad = {k: v.copy() for k, v in g.items()}
    worst = int(o["rank"][-1])
    victim = int(cs[0])
    bad["label"][bad["label"] == victim] = worst
    bad["label"][worst] = worst
    with pytest.raises(AssertionError):
        _check(w, f, p, bad)


def test_quota_band_check_accepts_and_rejects():
    n, ncl, budget = 200, 7, 60
    s = W.make_scores(3, 1, n, "lognormal")[0].astype(np.float64)
    label = W.make_labels(3, 1, n, ncl)[0]
    want, nc, quota = oracle.select_quota(s, label, budget)
    assert oracle_quota_band_check(s, label, want, budget, KNORM_RTOL) == 0
    # swap a kept token with a dropped one of the same cluster whose score is far from the cut: rejected
    c = label[want[0]]
    members = np.flatnonzero(label == c)
    dropped = np.setdiff1d(members, want)
    far = dropped[np.argmax(s[dropped])]
    bad = np.sort(np.append(want[1:], far))
    with pytest.raises(AssertionError):
        oracle_quota_band_check(s, label, bad, budget, KNORM_RTOL)
    # the same swap is accepted once the two scores sit inside the band at the cut
    s2 = s.copy()
    kept_c = np.intersect1d(members, want)
    last_in = kept_c[np.argmax(s2[kept_c])]
    first_out = dropped[np.argmin(s2[dropped])]
    s2[first_out] = s2[last_in] * (1 + 1e-7)
    want2, _, _ = oracle.select_quota(s2, label, budget)
    swapped = np.sort(np.append(np.setdiff1d(want2, [last_in]), first_out))
    assert oracle_quota_band_check(s2, label, swapped, budget, KNORM_RTOL) == 2
