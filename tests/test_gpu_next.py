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


@pytest.mark.parametrize("n,clusters,keep_p", [(16384, 820, 0.06), (16384, 16384, 0.5), (9000, 3, 0.0), (1025, 1025, 0.2),
                                               (31, 5, 0.3), (1, 1, 0.0)])
def test_merge_planner_sizes(n, clusters, keep_p):
    """The planner at the largest span, with every token its own cluster, with a few huge clusters, and at sizes around
    its row (32) and pass (1024) granularity; labels are arbitrary token indices, one of them out of range."""
    rng = np.random.default_rng(n + clusters)
    B, Dh, vs = 2, 64, 3
    hid = W.f32_to_bf16_bits(rng.standard_normal((B, n + vs + 2, Dh)).astype(np.float32))
    ids = np.sort(rng.choice(n, size=clusters, replace=False)).astype(np.int32)
    label = ids[rng.integers(0, clusters, size=(B, n))]
    keep = (rng.random((B, n)) < keep_p).astype(np.uint8)
    vl = np.array([n, max(0, n - 7)], dtype=np.int32)
    label[1, : vl[1]] = np.minimum(label[1, : vl[1]], max(vl[1] - 1, 0))      # labels stay inside the sample's own span
    _check_merge(hid, vs, vl, label, keep, min(n, 900))


def test_merge_label_out_of_range_is_clamped():
    rng = np.random.default_rng(11)
    n, Dh = 100, 64
    hid = W.f32_to_bf16_bits(rng.standard_normal((1, n, Dh)).astype(np.float32))
    label = rng.integers(0, 7, size=(1, n)).astype(np.int32)
    bad = label.copy()
    bad[0, 5], bad[0, 50] = 10 ** 6, -3
    ref = label.copy()
    ref[0, 5] = ref[0, 50] = n - 1
    keep = np.zeros((1, n), np.uint8)
    a = _gpu_merge(hid, 0, n, bad, keep, n)
    b = _gpu_merge(hid, 0, n, ref, keep, n)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)


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


# shapes: a row on 8 / 16 / 32 lanes (d up to 64 / 128 / 256), rows longer than 32 pieces (d = 264, 512), one key
# only, more heads than the second kernel has warps, key counts around the chunk (256) and block (64) sizes
@pytest.mark.parametrize("B,H,M,d", [(2, 4, 33, 16), (1, 1, 2, 8), (3, 16, 577, 64), (2, 12, 1300, 128),
                                     (2, 3, 300, 256), (1, 2, 70, 264), (1, 2, 257, 512), (2, 5, 1, 64),
                                     (1, 19, 256, 72), (1, 40, 65, 32), (1, 2, 4100, 128)])
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
        assert S[b].shape == want.shape
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


# ======================================================================================= K projection + K-norm
# The call writes K in bf16 and reports Eq. 4 of exactly those values.  What is checked:
#   K:      |gpu - oracle fp64| <= one bf16 spacing of the value (2^-8 relative: the rounding step, taken on an fp32
#           accumulator here and on the fp64 value in the oracle, may fall either way near a tie) + the fp32
#           accumulation error, bounded by 2e-6 |x_t| |w_c|; and nearly all elements round to the oracle's bits;
#   score:  relative 1e-5 against Eq. 4 of the K the call wrote (the definition of what it reports), and relative
#           1e-4 against the oracle's own rounded K (a few roundings that fell the other way move it by ~1e-5).
KPROJ_ULP = 2.0 ** -8


def _kproj_case(B, N, Dh, H, d, rope, vis_start, Nv, rows=None, seed=0):
    rng = np.random.default_rng(seed)
    hid = W.f32_to_bf16_bits(rng.standard_normal((B, N, Dh)).astype(np.float32))
    Wk = W.f32_to_bf16_bits((rng.standard_normal((H * d, Dh)) / np.sqrt(Dh)).astype(np.float32))
    n_pos = N + 5
    cos = sin = pos = None
    if rope:
        inv = 1.0 / (10000.0 ** (np.arange(d // 2) / (d // 2)))
        ang = np.arange(n_pos)[:, None] * inv[None, :]
        cos, sin = np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)
        pos = rng.integers(0, n_pos, size=(B, N)).astype(np.int32)
    K_out = torch.zeros((B, H, N, d), dtype=torch.bfloat16, device=DEV)
    score = torch.full((B, Nv), -7.0, dtype=torch.float32, device=DEV)
    ws = vb.alloc_workspace(vb.OP_KPROJ, B=B, H=H, N=N, d=d)
    t = lambda a: None if a is None else torch.from_numpy(a).to(DEV)
    vb.vitcop_kproj_knorm(vb.bf16_tensor(hid), vb.bf16_tensor(Wk), H, d, K_out, ws, vis_start=vis_start, score=score,
                          rope_cos=t(cos), rope_sin=t(sin), position_ids=t(pos))
    assert vb.vitcop_poll_status(ws) == vb.OK
    g_K, g_score = vb.bf16_bits(K_out), score.cpu().numpy()
    # Eq. 4 of the K that was written, every token of the span
    own = oracle.knorm(g_K, vis_start, Nv)
    assert np.all(rel_err(g_score, own) <= KNORM_RTOL), rel_err(g_score, own).max()
    # against the oracle's projection: all rows of small cases, a seeded sample of rows otherwise
    xf, wf = W.bf16_bits_to_f32(hid).astype(np.float64), W.bf16_bits_to_f32(Wk).astype(np.float64)
    wn = np.sqrt((wf * wf).sum(1)).reshape(H, 1, d)
    same = total = 0
    for b in range(B):
        sel = np.arange(N) if rows is None else np.sort(rng.permutation(N)[:rows])
        K64, Kb, o_score = oracle.kproj_knorm(np.ascontiguousarray(hid[b, sel]), Wk, H, d,
                                              None if cos is None else cos.astype(np.float64),
                                              None if sin is None else sin.astype(np.float64),
                                              None if pos is None else np.ascontiguousarray(pos[b, sel]))
        if pos is None and rope:
            raise AssertionError
        got = W.bf16_bits_to_f32(g_K[b][:, sel]).astype(np.float64)
        xn = np.sqrt((xf[b, sel] ** 2).sum(1)).reshape(1, -1, 1)
        assert np.all(np.abs(got - K64) <= KPROJ_ULP * np.abs(K64) + 2e-6 * xn * wn)
        same += int((g_K[b][:, sel] == Kb).sum())
        total += Kb.size
        in_span = (sel >= vis_start) & (sel < vis_start + Nv)
        if in_span.any():
            assert np.all(rel_err(g_score[b, sel[in_span] - vis_start], o_score[in_span]) <= 1e-4)
    assert same >= 0.97 * total, (same, total)


@pytest.mark.parametrize("B,N,Dh,H,d,rope", [(2, 77, 128, 3, 64, False), (1, 300, 256, 4, 128, True),
                                              (3, 130, 192, 2, 256, True), (2, 64, 64, 5, 32, False),
                                              (2, 200, 320, 6, 64, True), (1, 129, 64, 1, 128, False)])
def test_kproj_knorm_small(B, N, Dh, H, d, rope):
    _kproj_case(B, N, Dh, H, d, rope, vis_start=min(5, N - 1), Nv=max(1, N - 9), seed=N)


def test_kproj_knorm_identity_weights_and_text_only_span():
    # W = I: K is the hidden row cut into heads, bit for bit, and the score is Eq. 4 of the input
    rng = np.random.default_rng(3)
    B, N, H, d = 2, 70, 2, 64
    hid = W.f32_to_bf16_bits(rng.standard_normal((B, N, H * d)).astype(np.float32))
    K_out = torch.zeros((B, H, N, d), dtype=torch.bfloat16, device=DEV)
    score = torch.zeros((B, N), dtype=torch.float32, device=DEV)
    ws = vb.alloc_workspace(vb.OP_KPROJ, B=B, H=H, N=N, d=d)
    eye = W.f32_to_bf16_bits(np.eye(H * d, dtype=np.float32))
    vb.vitcop_kproj_knorm(vb.bf16_tensor(hid), vb.bf16_tensor(eye), H, d, K_out, ws, score=score)
    want = np.ascontiguousarray(hid.reshape(B, N, H, d).transpose(0, 2, 1, 3))
    assert np.array_equal(vb.bf16_bits(K_out), want)
    assert np.all(rel_err(score.cpu().numpy(), oracle.knorm(want, 0, N)) <= KNORM_RTOL)
    vb.vitcop_kproj_knorm(vb.bf16_tensor(hid), vb.bf16_tensor(eye), H, d, K_out, ws)          # no span: K only
    assert vb.vitcop_poll_status(ws) == vb.OK and np.array_equal(vb.bf16_bits(K_out), want)


@pytest.mark.parametrize("name", ["c1", "c4"])
def test_kproj_knorm_workload_shapes(name):
    """The projection at the shapes of a benchmark workload (c1: 10240 tokens x 4096 -> 32 heads of 128); the oracle
    checks a seeded sample of token rows, Eq. 4 of the written K is checked on every token."""
    w = W.workload(name)
    _kproj_case(w.B, w.N, w.Dh, w.H, w.d, True, w.vis_start, w.Nv, rows=6, seed=1)
