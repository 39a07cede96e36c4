"""Parity at the full sizes of the five benchmark workloads, in the launch configuration bench.py times.

K-norm, selection and compaction are compared on every element (the oracle handles them in seconds).
The filter is compared on every token for c0-c3; for c4 (16384 tokens, 1.4 TFLOP of fp64 per sample on
the CPU) one sample is checked in full and the similarity scores on a seeded sample of rows.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_17818_b200 import binding as vb
from paper_2601_17818_b200 import workloads as W

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from gpu_helpers import (KNORM_RTOL, SIM_ATOL, check_vic_sample, gpu_filter, gpu_knorm, gpu_similarity_rows,
                             rel_err)
    from test_gpu_parity import _run_chain


@pytest.mark.parametrize("name", ["c0", "c1", "c2", "c3", "c4"])
def test_knorm_full(name):
    w = W.workload(name)
    K, _ = W.make_kv(w, 0, w.Nv)
    got = gpu_knorm(K, w.vis_start, w.Nv)
    want = oracle.knorm(K, w.vis_start, w.Nv)
    assert got.shape == want.shape == (w.B, w.Nv)
    assert np.all(rel_err(got, want) <= KNORM_RTOL)


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4"])
def test_prune_chain_full(name):
    stats = _run_chain(W.workload(name))
    print("chain", name, stats)


@pytest.mark.parametrize("name", ["c1", "c2", "c3"])
def test_filter_full(name):
    w = W.workload(name)
    f = W.make_features(w)
    p = W.make_positions(w)
    g = gpu_filter(f, p, 0, w.d_c, w.tau, w.n_centers)
    assert g.status == vb.OK and np.all(g.n_clusters == w.n_centers)
    rep = []
    samples = range(w.B) if name == "c1" else (0, w.B - 1)
    for b in samples:
        check_vic_sample(f[b], p[b], 0, w.d_c, w.tau, w.n_centers, g.rho[b], g.delta2[b], g.parent[b], g.label[b], rep)
    print("filter", name, rep)
    # similarity scores themselves, all rows of one sample
    b = w.B - 1
    got = gpu_similarity_rows(f[b:b + 1], 0, 0, w.Nv)[0]
    _, sim = oracle.feature_distance(f[b], 0, want_d2=False)
    assert np.abs(got - sim).max() <= SIM_ATOL


def test_filter_full_c4():
    w = W.workload("c4")
    f = W.make_features(w)
    p = W.make_positions(w)
    g = gpu_filter(f, p, 0, w.d_c, w.tau, w.n_centers)
    assert g.status == vb.OK and np.all(g.n_clusters == w.n_centers)
    rep = []
    check_vic_sample(f[1], p[1], 0, w.d_c, w.tau, w.n_centers, g.rho[1], g.delta2[1], g.parent[1], g.label[1], rep)
    print("filter c4", rep)
    rows = np.sort(np.random.default_rng(0).permutation(w.Nv - 256)[:4])
    for r0 in rows:
        got = gpu_similarity_rows(f[0:1], 0, int(r0), int(r0) + 64)[0]
        _, sim = oracle.feature_distance(f[0], 0, rows=(int(r0), int(r0) + 64), want_d2=False)
        assert np.abs(got - sim).max() <= SIM_ATOL
    # the other sample: invariants that hold at any size
    lab = g.label[0]
    cs = np.flatnonzero(lab == np.arange(w.Nv))
    assert len(cs) == w.n_centers and set(np.unique(lab).tolist()) == set(cs.tolist())
    par = g.parent[0]
    ok = par >= 0
    rho = g.rho[0]
    assert np.all((rho[par[ok]] > rho[ok]) | ((rho[par[ok]] == rho[ok]) & (par[ok] < np.flatnonzero(ok))))
