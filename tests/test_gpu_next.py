"""GPU-vs-oracle parity of the stages around the core chain: cluster merge (Eq. 6) and Stage I saliency (Eq. 1)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_17818_b200 import binding as vb
from paper_2601_17818_b200 import workloads as W

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from gpu_helpers import DEV, KNORM_RTOL, dev_i32, gpu_filter, gpu_select, oracle_band_check, rel_err

MERGE_RTOL = 1e-5        # merged rows: |gpu - oracle| <= 1e-5 * mean_i |t_i| over the averaged rows (fp32 sums vs fp64)
SAL_RTOL = 1e-5          # saliency: relative


def _gpu_merge(hid_bits, vis_start, vis_len, label, keep_mask, Mcap):
    hid = vb.bf16_tensor(hid_bits)
    B, N, Dh = hid.shape
    lab = dev_i32(label)
    km = torch.from_numpy(np.ascontiguousarray(keep_mask, dtype=np.uint8)).to(DEV)
    mb = torch.zeros((B, Mcap, Dh), dtype=torch.bfloat16, device=DEV)
    mf = torch.full((B, Mcap, Dh), -7.0, dtype=torch.float32, device=DEV)
    ml = torch.full((B, Mcap), -7, dtype=torch.int32, device=DEV)
    mc = torch.full((B, Mcap), -7, dtype=torch.int32, device=DEV)
    nm = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    vl = int(vis_len) if np.isscalar(vis_len) else dev_i32(vis_len)
    ws = vb.alloc_workspace(vb.OP_MERGE, B=B, Nv=lab.shape[1], N=Mcap)
    vb.vitcop_merge_clusters(hid, vis_start, vl, lab, km, ml, mc, nm, ws, merged=mb, merged_f32=mf)
    torch.cuda.synchronize()
    return vb.bf16_bits(mb), mf.cpu().numpy(), ml.cpu().numpy(), mc.cpu().numpy(), nm.cpu().numpy()


def _check_merge(hid_bits, vis_start, vis_len, label, keep_mask, Mcap):
    B = hid_bits.shape[0]
    mb, mf, ml, mc, nm = _gpu_merge(hid_bits, vis_start, vis_len, label, keep_mask, Mcap)
    for b in range(B):
        n = int(vis_len) if np.isscalar(vis_len) else int(vis_len[b])
        want, wl, wc = oracle.merge_clusters(hid_bits[b], vis_start, label[b, :n], keep_mask[b, :n])
        assert nm[b] == len(wl)
        m = min(len(wl), Mcap)
        assert np.array_equal(ml[b, :m], wl[:m]) and np.array_equal(mc[b, :m], wc[:m])
        x = np.abs(W.bf16_bits_to_f32(hid_bits[b, vis_start:vis_start + n]).astype(np.float64))
        for r in range(m):
            members = (label[b, :n] == wl[r]) & (keep_mask[b, :n] == 0)
            scale = x[members].mean(0)
            assert np.all(np.abs(mf[b, r] - want[r]) <= MERGE_RTOL * scale + 1e-30)
        # the bf16 rows are the kernel's own fp32 averages rounded to nearest even, bit for bit
        assert np.array_equal(mb[b, :m], W.f32_to_bf16_bits(mf[b, :m]))
        assert np.all(mf[b, m:] == -7.0) and np.all(ml[b, m:] == -7)          # rows past n_merged stay untouched


def test_merge_small_and_edges():
    rng = np.random.default_rng(4)
    B, N, Dh, vs, n = 3, 75, 64, 5, 60
    hid = W.f32_to_bf16_bits(rng.standard_normal((B, N, Dh)).astype(np.float32))
    label = W.make_labels(2, B, n, 6)
    keep = (rng.random((B, n)) < 0.4).astype(np.uint8)
    keep[1] = 1                                               # every token kept: no merged row at all
    keep[2] = 0                                               # nothing kept: every cluster averages all its tokens
    _check_merge(hid, vs, n, label, keep, n)
    # ragged spans, one of them empty; capacity below the number of clusters
    vl = np.array([60, 17, 0], dtype=np.int32)
    lab2 = label.copy()
    lab2[1, :17] = W.make_labels(3, 1, 17, 4)[0]
    keep2 = (rng.random((B, n)) < 0.3).astype(np.uint8)
    _check_merge(hid, vs, vl, lab2, keep2, n)
    _check_merge(hid, vs, n, label, np.zeros((B, n), np.uint8), 2)
    # one giant cluster (all labels equal) with a hidden size that spans several CTA slices
    hid = W.f32_to_bf16_bits(rng.standard_normal((1, 700, 4096)).astype(np.float32))
    _check_merge(hid, 0, 700, np.zeros((1, 700), np.int32), (rng.random((1, 700)) < 0.1).astype(np.uint8), 4)


@pytest.mark.parametrize("name", ["tiny", "c0"])
def test_stage_two_with_merge(name):
    """Stage II as Algorithm 3 states it: VIC labels -> K-norm quota elites -> merged token per cluster."""
    w = W.workload(name)
    f, p = W.make_features(w), W.make_positions(w)
    g = gpu_filter(f, p, 0, w.d_c, w.tau, w.n_centers)
    K, _ = W.make_kv(w, 0, w.Nv)
    score = oracle.knorm(K, w.vis_start, w.Nv).astype(np.float32)
    budget = w.budgets[0]
    keeps, nk, mask, status = gpu_select(score, budget, label=g.label)
    assert status == vb.OK
    hid = W.make_hidden(w)
    _check_merge(hid, w.vis_start, w.Nv, g.label, mask, w.n_centers)
    _, _, ml, mc, nm = _gpu_merge(hid, w.vis_start, w.Nv, g.label, mask, w.n_centers)
    for b in range(w.B):
        # elites + merged tokens never exceed the budget (Algorithm 3), every non-elite token is merged once
        assert nk[b] + nm[b] <= budget
        assert mc[b, :nm[b]].sum() == w.Nv - nk[b]


@pytest.mark.parametrize("B,H,M,d", [(2, 4, 33, 16), (1, 1, 2, 8), (3, 16, 577, 64), (2, 12, 1300, 128)])
def test_cls_saliency(B, H, M, d):
    q, K = W.make_cls_qk(M, B, H, M, d)
    scale = 1.0 / np.sqrt(d)
    S = torch.full((B, M - 1), -7.0, dtype=torch.float32, device=DEV)
    c = torch.full((B,), -7.0, dtype=torch.float32, device=DEV)
    ws = vb.alloc_workspace(vb.OP_SALIENCY, B=B, H=H, N=M)
    vb.vitcop_cls_saliency(vb.bf16_tensor(q), vb.bf16_tensor(K), scale, S, ws, cls_self=c)
    torch.cuda.synchronize()
    S, c = S.cpu().numpy(), c.cpu().numpy()
    for b in range(B):
        want, wc = oracle.cls_saliency(q[b], K[b], scale)
        assert np.all(rel_err(S[b], want) <= SAL_RTOL) and abs(c[b] - wc) <= SAL_RTOL * wc
        assert abs(S[b].sum() + c[b] - H) <= 1e-4             # every head's attention row sums to one


def test_stage_one_chain():
    """Stage I of Algorithm 1 on CLIP-shaped inputs: saliency -> keep the floor(m * pi_1) largest -> compact features."""
    B, H, M, d, D = 4, 16, 577, 64, 1024
    m = M - 1
    q, K = W.make_cls_qk(0, B, H, M, d)
    scale = 1.0 / np.sqrt(d)
    S = torch.empty((B, m), dtype=torch.float32, device=DEV)
    ws = vb.alloc_workspace(vb.OP_SALIENCY, B=B, H=H, N=M)
    vb.vitcop_cls_saliency(vb.bf16_tensor(q), vb.bf16_tensor(K), scale, S, ws)
    k1 = vb.vitcop_stage_count(m, 0.3)
    assert k1 == oracle.stage_count(m, 0.3) == 172
    g_S = S.cpu().numpy()
    keeps, nk, mask, _ = gpu_select(g_S, k1, largest=True)
    rng = np.random.default_rng(1)
    feat = rng.integers(0, 65536, size=(B, m, D)).astype(np.uint16)
    tf = vb.bf16_tensor(feat)
    out = torch.zeros((B, k1, D), dtype=torch.bfloat16, device=DEV)
    olen = torch.zeros((B,), dtype=torch.int32, device=DEV)
    ki = np.stack(keeps).astype(np.int32)
    vb.vitcop_compact_kv(tf, None, None, 0, m, dev_i32(ki), dev_i32(nk), out, None, None, olen)
    got = vb.bf16_bits(out)
    for b in range(B):
        want_S, _ = oracle.cls_saliency(q[b], K[b], scale)
        oracle_band_check(want_S, keeps[b], k1, SAL_RTOL, largest=True)
        assert np.array_equal(keeps[b], oracle.select_plain(g_S[b].astype(np.float64), k1, True))
        assert np.array_equal(got[b], feat[b][keeps[b]]) and int(olen[b]) == k1
