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


# Stage II through the one call the benchmark times, compared DIRECTLY with the oracle: K-norm scores (computed in
# part by the side warps of the one-kernel sweep on c0/c1, by the stand-alone kernel elsewhere), the clustering by
# the three-level rule, the quota selection and the compacted rows.
@pytest.mark.parametrize("name,samples", [("tiny", None), ("c0", None), ("c1", None), ("c2", (7,)), ("c3", (3,)),
                                          ("c4", (1,))])
def test_collaborative_step_vs_oracle(name, samples):
    from gpu_helpers import DEV, oracle_quota_band_check
    w = W.workload(name)
    B, n = w.B, w.Nv
    f, p = W.make_features(w), W.make_positions(w)
    K_b, V_b = W.make_kv(w, 0, n)
    hid_b = W.make_hidden(w)
    budget = w.budgets[0]
    Ncap = w.T + budget
    z = lambda *s, dt: torch.zeros(s, dtype=dt, device=DEV)
    ho, Ko, Vo = (z(B, Ncap, w.Dh, dt=torch.bfloat16), z(B, w.H, Ncap, w.d, dt=torch.bfloat16),
                  z(B, w.H, Ncap, w.d, dt=torch.bfloat16))
    olen, kpos = z(B, dt=torch.int32), z(B, Ncap, dt=torch.int32)
    label, ncl = z(B, n, dt=torch.int32), z(B, dt=torch.int32)
    rho, d2, par = z(B, n, dt=torch.float32), z(B, n, dt=torch.float32), z(B, n, dt=torch.int32)
    score, kidx, nkeep = z(B, n, dt=torch.float32), z(B, n, dt=torch.int32), z(B, dt=torch.int32)
    ws = vb.alloc_workspace(vb.OP_COLLAB_STEP, B=B, Nv=n, D=w.D)
    vb.vitcop_collaborative_step(vb.bf16_tensor(f), torch.from_numpy(p.copy()).to(DEV), vb.bf16_tensor(hid_b),
                                 vb.bf16_tensor(K_b), vb.bf16_tensor(V_b), w.vis_start, budget, ho, Ko, Vo, olen, label,
                                 ncl, ws, metric=0, d_c=w.d_c, tau=w.tau, n_centers=w.n_centers, kept_pos=kpos,
                                 score_out=score, keep_idx_out=kidx, n_keep_out=nkeep, rho=rho, delta2=d2, parent=par)
    assert vb.vitcop_poll_status(ws) == vb.OK
    g_score, g_idx, g_nk = score.cpu().numpy(), kidx.cpu().numpy(), nkeep.cpu().numpy()
    g_label, g_rho, g_d2, g_par = label.cpu().numpy(), rho.cpu().numpy(), d2.cpu().numpy(), par.cpu().numpy()
    g_ho, g_Ko, g_Vo = vb.bf16_bits(ho), vb.bf16_bits(Ko), vb.bf16_bits(Vo)
    g_olen, g_pos = olen.cpu().numpy(), kpos.cpu().numpy()
    assert np.all(ncl.cpu().numpy() == w.n_centers)
    # Eq. 4
    o_score = oracle.knorm(K_b, w.vis_start, n)
    assert np.all(rel_err(g_score, o_score) <= KNORM_RTOL)
    # Algorithm 2
    rep = []
    for b in (range(B) if samples is None else samples):
        check_vic_sample(f[b], p[b], 0, w.d_c, w.tau, w.n_centers, g_rho[b], g_d2[b], g_par[b], g_label[b], rep)
    print("collaborative step", name, rep)
    diffs = 0
    for b in range(B):
        keep = g_idx[b, : g_nk[b]]
        # Eq. 5 / Algorithm 3: exact on the kernel's own fp32 scores; vs the oracle's scores up to the band at each cut
        want, nc, _ = oracle.select_quota(g_score[b].astype(np.float64), g_label[b], budget)
        assert nc == w.n_centers and np.array_equal(keep, want)
        diffs += oracle_quota_band_check(o_score[b], g_label[b], keep, budget, KNORM_RTOL)
        # compaction: bit-exact rows
        o = oracle.compact(hid_b[b], K_b[b], V_b[b], w.N, w.vis_start, n, keep, Ncap)
        L = o["out_len"]
        assert g_olen[b] == L == w.T + g_nk[b]
        assert np.array_equal(g_pos[b, :L], o["kept_pos"][:L])
        assert np.array_equal(g_ho[b, :L], o["hidden"][:L])
        assert np.array_equal(g_Ko[b, :, :L], o["K"][:, :L]) and np.array_equal(g_Vo[b, :, :L], o["V"][:, :L])
    print("collaborative step", name, "selection differences inside the band:", diffs)
