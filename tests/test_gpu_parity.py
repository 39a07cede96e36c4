"""GPU-vs-oracle parity of the whole pruning chain, through the C ABI (``-m gpu``)."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2601_17818_b200 import binding as vb
from paper_2601_17818_b200 import workloads as W

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from gpu_helpers import (DEV, GRAM_RTOL, KNORM_RTOL, SIM_ATOL, check_vic_sample,
                             dev_i32, gpu_filter, gpu_knorm, gpu_select, gpu_similarity_rows, oracle_band_check,
                             oracle_quota_band_check, rel_err)


# ======================================================================================= K-norm (Eq. 4)
@pytest.mark.parametrize("shape", [(1, 1, 5, 8), (2, 3, 37, 64), (3, 8, 130, 128), (2, 4, 77, 256), (1, 2, 33, 24)])
@pytest.mark.parametrize("vis_start", [0, 3])
def test_knorm_small(shape, vis_start):
    B, H, N, d = shape
    rng = np.random.default_rng(N)
    K = W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32) * 3)
    nv = N - vis_start - 1
    got = gpu_knorm(K, vis_start, nv)
    want = oracle.knorm(K, vis_start, nv)
    assert np.all(rel_err(got, want) <= KNORM_RTOL)


def test_knorm_closed_forms_and_ragged():
    K = W.f32_to_bf16_bits(np.ones((2, 32, 40, 128), dtype=np.float32))
    assert np.array_equal(gpu_knorm(K, 0, 40), np.full((2, 40), 64.0, dtype=np.float32))
    rng = np.random.default_rng(0)
    K = W.f32_to_bf16_bits(rng.standard_normal((3, 4, 50, 64)).astype(np.float32))
    vl = np.array([0, 17, 45], dtype=np.int32)
    got = gpu_knorm(K, 5, vl, Nv_cap=45)
    want = oracle.knorm(K, 5, vl)
    for b in range(3):
        assert np.all(rel_err(got[b, :vl[b]], want[b, :vl[b]]) <= KNORM_RTOL)
        assert np.all(got[b, vl[b]:] == -7.0)             # entries past vis_len stay untouched
    # zeros, one-hot
    Kz = np.zeros((1, 2, 9, 16), dtype=np.float32)
    Kz[0, 1, 4, 3] = -2.5
    got = gpu_knorm(W.f32_to_bf16_bits(Kz), 0, 9)[0]
    assert got[4] == 2.5 and np.all(np.delete(got, 4) == 0)


def test_knorm_device_length_beyond_capacity_is_clamped():
    # a device-side length larger than the score row's capacity: only `capacity` tokens are scored, the next
    # sample's row and the memory behind the last row stay untouched
    rng = np.random.default_rng(4)
    B, H, N, d, cap = 2, 2, 64, 64, 21                    # 16 tokens per CTA: the capacity ends inside a CTA
    K = W.f32_to_bf16_bits(rng.standard_normal((B, H, N, d)).astype(np.float32))
    buf = torch.full((B + 1, cap), -7.0, dtype=torch.float32, device=DEV)
    vb.vitcop_knorm_score(vb.bf16_tensor(K), 3, dev_i32([40, 33]), buf[:B])
    torch.cuda.synchronize()
    got = buf.cpu().numpy()
    want = oracle.knorm(K, 3, cap)
    assert np.all(rel_err(got[:B], want) <= KNORM_RTOL)
    assert np.all(got[B] == -7.0)


def test_knorm_strided_view():
    # K stored [B, N, H, d] and viewed as [B, H, N, d]: the strides are arguments of the call
    rng = np.random.default_rng(1)
    raw = W.f32_to_bf16_bits(rng.standard_normal((2, 21, 5, 64)).astype(np.float32))
    Kt = vb.bf16_tensor(raw).permute(0, 2, 1, 3)
    score = torch.zeros((2, 21), dtype=torch.float32, device=DEV)
    vb.vitcop_knorm_score(Kt, 0, 21, score)
    want = oracle.knorm(np.ascontiguousarray(raw.transpose(0, 2, 1, 3)), 0, 21)
    assert np.all(rel_err(score.cpu().numpy(), want) <= KNORM_RTOL)


# ======================================================================================= selection
SIZES = [1, 2, 3, 7, 31, 32, 33, 129, 577, 1025, 5000, 16384]


@pytest.mark.parametrize("kind", ["lognormal", "ties", "equal", "signed"])
def test_select_plain_exact(kind):
    """Given identical fp32 scores the kept set is unique, so it must match bit for bit."""
    for n in SIZES:
        score = W.make_scores(n, 2, n, kind)
        for k in sorted({0, 1, n // 3, n - 1, n, n + 5}):
            if k < 0:
                continue
            for largest in ([False, True] if n <= 1025 else [False]):
                keeps, nk, mask, status = gpu_select(score, k, largest=largest)
                assert status == vb.OK
                for b in range(2):
                    want = oracle.select_plain(score[b].astype(np.float64), k, largest)
                    assert nk[b] == len(want)
                    assert np.array_equal(keeps[b], want), (n, k, kind, largest)
                    m = np.zeros(n, dtype=np.uint8)
                    m[want] = 1
                    assert np.array_equal(mask[b], m)


def test_select_nan_inf_and_signed_zero():
    s = np.array([[2.0, np.nan, 1.0, np.inf, 0.0, -0.0, -np.inf, 5.0]], dtype=np.float32)
    for k in range(0, 9):
        keeps, nk, _, _ = gpu_select(s, k)
        assert np.array_equal(keeps[0], oracle.select_plain(s[0].astype(np.float64), k))
        keeps, nk, _, _ = gpu_select(s, k, largest=True)
        assert np.array_equal(keeps[0], oracle.select_plain(s[0].astype(np.float64), k, True))


def test_select_ragged_lengths():
    cap = 300
    score = W.make_scores(7, 4, cap, "lognormal")
    vl = np.array([0, 1, 150, 300], dtype=np.int32)
    keeps, nk, mask, _ = gpu_select(score, 40, vis_len=vl)
    for b in range(4):
        want = oracle.select_plain(score[b, :vl[b]].astype(np.float64), 40)
        assert np.array_equal(keeps[b], want)
        assert np.all(mask[b, vl[b]:] == 7)               # mask past the span is untouched


# Even cluster sizes take the per-cluster rank search; a dominant cluster (skew) takes the sort below 4096 tokens and
# the per-cluster radix search above; more than 1024 clusters always take the sort.
@pytest.mark.parametrize("kind", ["lognormal", "ties", "equal"])
@pytest.mark.parametrize("skew", [0.0, 0.7])
def test_select_quota_exact(kind, skew):
    cases = [(1, 1), (10, 2), (97, 7), (576, 29), (1000, 1000), (2880, 144), (16384, 820),
             (4097, 3), (5000, 40), (6000, 1024), (8192, 2000)]
    if skew:
        cases = [(97, 7), (576, 29), (2880, 144), (4097, 3), (5000, 40), (6000, 1024), (16384, 820), (16384, 2)]
    for n, ncl in cases:
        score = W.make_scores(n + 1, 2, n, kind)
        label = W.make_labels(n, 2, n, ncl, skew=skew)
        for budget in sorted({ncl, ncl + 1, (n + ncl) // 2, n}):
            keeps, nk, mask, status = gpu_select(score, budget, label=label)
            assert status == vb.OK
            for b in range(2):
                want, nc, _ = oracle.select_quota(score[b].astype(np.float64), label[b], budget)
                assert nc == ncl
                assert np.array_equal(keeps[b], want), (n, ncl, budget, kind, skew)
                assert nk[b] + nc <= budget
        if ncl > 1:                                        # budget below the cluster count: device-side status
            keeps, nk, _, status = gpu_select(score, ncl - 1, label=label)
            assert status == vb.ERR_BUDGET and np.all(nk == 0)


@pytest.mark.parametrize("n,ncl,skew", [(64, 5, 0.0), (600, 20, 0.7), (5000, 40, 0.0), (5000, 40, 0.7)])
def test_select_quota_special_values(n, ncl, skew):
    """NaN (ranked after everything), infinities, signed zeros and many exact ties, through each search strategy."""
    rng = np.random.default_rng(n + ncl)
    score = rng.integers(0, 12, size=(2, n)).astype(np.float32)          # heavy ties
    special = np.array([np.nan, np.inf, -np.inf, 0.0, -0.0], dtype=np.float32)
    hit = rng.random((2, n)) < 0.1
    score[hit] = special[rng.integers(0, len(special), size=int(hit.sum()))]
    label = W.make_labels(n + 3, 2, n, ncl, skew=skew)
    for budget in (ncl + 1, (n + ncl) // 3, n):
        keeps, nk, _, status = gpu_select(score, budget, label=label)
        assert status == vb.OK
        for b in range(2):
            want, nc, _ = oracle.select_quota(score[b].astype(np.float64), label[b], budget)
            assert np.array_equal(keeps[b], want), (n, ncl, skew, budget)


# ======================================================================================= compaction
def _rand_bits(rng, shape):
    return rng.integers(0, 65536, size=shape).astype(np.uint16)


def _gpu_compact(hid, K, V, vis_start, vis_len, keeps, Ncap, seq_len=None):
    B = (K if K is not None else hid).shape[0]
    th = None if hid is None else vb.bf16_tensor(hid)
    tK = None if K is None else vb.bf16_tensor(K)
    tV = None if V is None else vb.bf16_tensor(V)
    stride = max(1, max(len(k) for k in keeps))
    ki = np.full((B, stride), -1, dtype=np.int32)
    for b, k in enumerate(keeps):
        ki[b, :len(k)] = k
    nk = dev_i32([len(k) for k in keeps])
    ho = None if hid is None else torch.zeros((B, Ncap, hid.shape[2]), dtype=torch.bfloat16, device=DEV)
    Ko = None if K is None else torch.zeros((B, K.shape[1], Ncap, K.shape[3]), dtype=torch.bfloat16, device=DEV)
    Vo = None if V is None else torch.zeros((B, V.shape[1], Ncap, V.shape[3]), dtype=torch.bfloat16, device=DEV)
    pos = torch.full((B, Ncap), -7, dtype=torch.int32, device=DEV)
    olen = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    vl = int(vis_len) if np.isscalar(vis_len) else dev_i32(vis_len)
    sl = None if seq_len is None else dev_i32(seq_len)
    vb.vitcop_compact_kv(th, tK, tV, vis_start, vl, dev_i32(ki), nk, ho, Ko, Vo, olen, kept_pos=pos, seq_len=sl)
    torch.cuda.synchronize()
    f = lambda t: None if t is None else vb.bf16_bits(t)
    return f(ho), f(Ko), f(Vo), pos.cpu().numpy(), olen.cpu().numpy()


@pytest.mark.parametrize("B,H,N,d,Dh,vs,nv", [(1, 1, 9, 8, 8, 0, 9), (2, 3, 50, 64, 256, 7, 30), (3, 32, 140, 128, 4096, 64, 70),
                                              (2, 4, 77, 128, 3584, 5, 72)])
def test_compact_bit_exact(B, H, N, d, Dh, vs, nv):
    rng = np.random.default_rng(N)
    hid, K, V = _rand_bits(rng, (B, N, Dh)), _rand_bits(rng, (B, H, N, d)), _rand_bits(rng, (B, H, N, d))
    keeps = [np.sort(rng.permutation(nv)[: rng.integers(0, nv + 1)]).astype(np.int32) for _ in range(B)]
    keeps[0] = np.arange(nv, dtype=np.int32)              # keep-all sample
    if B > 1:
        keeps[1] = np.zeros(0, dtype=np.int32)            # keep-none sample
    Ncap = N
    ho, Ko, Vo, pos, olen = _gpu_compact(hid, K, V, vs, nv, keeps, Ncap)
    for b in range(B):
        o = oracle.compact(hid[b], K[b], V[b], N, vs, nv, keeps[b], Ncap)
        L = o["out_len"]
        assert olen[b] == L
        assert np.array_equal(pos[b], o["kept_pos"])
        assert np.array_equal(ho[b, :L], o["hidden"][:L])
        assert np.array_equal(Ko[b, :, :L], o["K"][:, :L]) and np.array_equal(Vo[b, :, :L], o["V"][:, :L])
        assert np.all(ho[b, L:] == 0) and np.all(Ko[b, :, L:] == 0)      # rows past out_len are never written


def test_compact_ragged_partial_tensors_and_small_capacity():
    rng = np.random.default_rng(3)
    B, H, N, d, Dh, vs = 3, 2, 40, 16, 32, 4
    hid, K, V = _rand_bits(rng, (B, N, Dh)), _rand_bits(rng, (B, H, N, d)), _rand_bits(rng, (B, H, N, d))
    vl = np.array([30, 10, 0], dtype=np.int32)
    sl = np.array([40, 20, 9], dtype=np.int32)
    keeps = [np.array([0, 5, 29], np.int32), np.array([9], np.int32), np.zeros(0, np.int32)]
    ho, Ko, Vo, pos, olen = _gpu_compact(hid, K, V, vs, vl, keeps, N, seq_len=sl)
    for b in range(B):
        o = oracle.compact(hid[b], K[b], V[b], sl[b], vs, vl[b], keeps[b], N)
        L = o["out_len"]
        assert olen[b] == L and np.array_equal(pos[b], o["kept_pos"])
        assert np.array_equal(ho[b, :L], o["hidden"][:L]) and np.array_equal(Vo[b, :, :L], o["V"][:, :L])
    # hidden only / K only
    ho, _, _, pos, olen = _gpu_compact(hid, None, None, vs, 30, [keeps[0]] * B, N)
    o = oracle.compact(hid[1], None, None, N, vs, 30, keeps[0], N)
    assert np.array_equal(ho[1, :o["out_len"]], o["hidden"][:o["out_len"]])
    _, Ko, _, pos, olen = _gpu_compact(None, K, None, vs, 30, [keeps[0]] * B, N)
    o = oracle.compact(None, K[2], None, N, vs, 30, keeps[0], N)
    assert np.array_equal(Ko[2, :, :o["out_len"]], o["K"][:, :o["out_len"]])
    # capacity smaller than the result: nothing past Ncap is written, out_len reports the full length
    ho, Ko, Vo, pos, olen = _gpu_compact(hid, K, V, vs, 30, [np.arange(30, dtype=np.int32)] * B, 12)
    assert np.all(olen == N)
    assert np.array_equal(ho[0], hid[0, :12]) and np.array_equal(Ko[0], K[0, :, :12])


# ======================================================================================= fused step
def _run_chain(w, B=None, use_labels=None, check_scores=True):
    """Successive vitcop_prune_step calls on a shrinking sequence vs the oracle chain.  Returns counts."""
    B = w.B if B is None else B
    hid0 = W.make_hidden(w, B=B)
    n_vis = w.Nv
    N = w.T + n_vis
    hid_dev = vb.bf16_tensor(hid0)
    hid_ref = [hid0[b] for b in range(B)]
    vis_len_dev = None
    seq_len_dev = None
    stats = dict(band_diffs=0, steps=0)
    for step, budget in enumerate(w.budgets):
        K, V = W.make_kv(w, step, n_vis, B=B)
        Ncur = w.T + n_vis
        tK, tV = vb.bf16_tensor(K), vb.bf16_tensor(V)
        th = hid_dev[:, :Ncur].contiguous()
        Ncap = w.T + min(budget, n_vis)
        ho = torch.zeros((B, Ncap, w.Dh), dtype=torch.bfloat16, device=DEV)
        Ko = torch.zeros((B, w.H, Ncap, w.d), dtype=torch.bfloat16, device=DEV)
        Vo = torch.zeros((B, w.H, Ncap, w.d), dtype=torch.bfloat16, device=DEV)
        olen = torch.zeros((B,), dtype=torch.int32, device=DEV)
        kpos = torch.zeros((B, Ncap), dtype=torch.int32, device=DEV)
        score = torch.zeros((B, n_vis), dtype=torch.float32, device=DEV)
        kidx = torch.zeros((B, n_vis), dtype=torch.int32, device=DEV)
        nkeep = torch.zeros((B,), dtype=torch.int32, device=DEV)
        ws = vb.alloc_workspace(vb.OP_PRUNE_STEP, B=B, Nv=n_vis)
        lab = None
        if use_labels is not None and step == 0:
            lab = dev_i32(use_labels)
        vb.vitcop_prune_step(th, tK, tV, w.vis_start, n_vis, n_vis, budget, ho, Ko, Vo, olen, ws, label=lab,
                             kept_pos=kpos, score_out=score, keep_idx_out=kidx, n_keep_out=nkeep)
        assert vb.vitcop_poll_status(ws) == vb.OK
        g_score, g_idx, g_nk = score.cpu().numpy(), kidx.cpu().numpy(), nkeep.cpu().numpy()
        g_ho, g_Ko, g_Vo = vb.bf16_bits(ho), vb.bf16_bits(Ko), vb.bf16_bits(Vo)
        g_olen, g_pos = olen.cpu().numpy(), kpos.cpu().numpy()
        o_score = oracle.knorm(K, w.vis_start, n_vis)
        if check_scores:
            assert np.all(rel_err(g_score, o_score) <= KNORM_RTOL)
        new_ref = []
        for b in range(B):
            keep_g = g_idx[b, :g_nk[b]]
            if lab is None:
                stats["band_diffs"] += oracle_band_check(o_score[b], keep_g, budget, KNORM_RTOL)
                assert g_nk[b] == min(budget, n_vis)
                # exact given the GPU's own fp32 scores
                assert np.array_equal(keep_g, oracle.select_plain(g_score[b].astype(np.float64), budget))
            else:
                # exact given the GPU's own fp32 scores; against the oracle's scores only tokens inside the
                # tolerance band at a cluster's cut may differ
                want, nc, _ = oracle.select_quota(g_score[b].astype(np.float64), use_labels[b], budget)
                assert np.array_equal(keep_g, want)
                stats["band_diffs"] += oracle_quota_band_check(o_score[b], np.asarray(use_labels[b]), keep_g, budget,
                                                               KNORM_RTOL)
            # compaction: byte-exact given the GPU's keep list
            o = oracle.compact(hid_ref[b], K[b], V[b], Ncur, w.vis_start, n_vis, keep_g, Ncap)
            L = o["out_len"]
            assert g_olen[b] == L == w.T + g_nk[b]
            assert np.array_equal(g_pos[b, :L], o["kept_pos"][:L])
            assert np.array_equal(g_ho[b, :L], o["hidden"][:L])
            assert np.array_equal(g_Ko[b, :, :L], o["K"][:, :L]) and np.array_equal(g_Vo[b, :, :L], o["V"][:, :L])
            new_ref.append(o["hidden"][:L].copy())
        if lab is not None:
            # quota mode keeps a per-sample count; continue the chain on the common prefix capacity
            n_next = int(g_nk.min())
            hid_ref = [r[: w.T + n_next] for r in new_ref]
            hid_dev = ho[:, : w.T + n_next].contiguous()
            n_vis = n_next
        else:
            hid_ref = new_ref
            hid_dev = ho
            n_vis = min(budget, n_vis)
        stats["steps"] += 1
    return stats


@pytest.mark.parametrize("name", ["tiny", "c0"])
def test_prune_step_chain_small(name):
    _run_chain(W.workload(name))


def test_prune_step_quota_with_random_labels():
    w = W.workload("tiny")
    labels = W.make_labels(5, w.B, w.Nv, w.n_centers)
    _run_chain(w, use_labels=labels)


def test_prune_step_ragged_device_lengths():
    """vis_len and seq_len as device arrays, text on both sides of the span."""
    rng = np.random.default_rng(11)
    B, H, N, d, Dh, vs = 3, 4, 120, 64, 128, 10
    K = W.f32_to_bf16_bits(rng.standard_normal((B, H, N, d)).astype(np.float32))
    V = _rand_bits(rng, (B, H, N, d))
    hid = _rand_bits(rng, (B, N, Dh))
    vl = np.array([100, 37, 1], dtype=np.int32)
    sl = np.array([120, 60, 30], dtype=np.int32)
    budget, cap = 20, 100
    Ncap = N
    ho = torch.zeros((B, Ncap, Dh), dtype=torch.bfloat16, device=DEV)
    Ko = torch.zeros((B, H, Ncap, d), dtype=torch.bfloat16, device=DEV)
    Vo = torch.zeros((B, H, Ncap, d), dtype=torch.bfloat16, device=DEV)
    olen = torch.zeros((B,), dtype=torch.int32, device=DEV)
    nkeep = torch.zeros((B,), dtype=torch.int32, device=DEV)
    kidx = torch.zeros((B, cap), dtype=torch.int32, device=DEV)
    ws = vb.alloc_workspace(vb.OP_PRUNE_STEP, B=B, Nv=cap)
    vb.vitcop_prune_step(vb.bf16_tensor(hid), vb.bf16_tensor(K), vb.bf16_tensor(V), vs, dev_i32(vl), cap, budget,
                         ho, Ko, Vo, olen, ws, seq_len=dev_i32(sl), keep_idx_out=kidx, n_keep_out=nkeep)
    assert vb.vitcop_poll_status(ws) == vb.OK
    g_ho, g_Ko = vb.bf16_bits(ho), vb.bf16_bits(Ko)
    for b in range(B):
        s = oracle.knorm(K[b:b + 1], vs, int(vl[b]))[0]
        keep = kidx.cpu().numpy()[b, : nkeep.cpu().numpy()[b]]
        oracle_band_check(s, keep, budget, KNORM_RTOL)
        o = oracle.compact(hid[b], K[b], V[b], sl[b], vs, vl[b], keep, Ncap)
        L = o["out_len"]
        assert olen.cpu().numpy()[b] == L
        assert np.array_equal(g_ho[b, :L], o["hidden"][:L]) and np.array_equal(g_Ko[b, :, :L], o["K"][:, :L])


def test_prune_step_text_only_batch():
    """No visual tokens at all: nothing is scored or selected, every row is copied, the lengths stay."""
    rng = np.random.default_rng(12)
    B, H, N, d, Dh = 2, 2, 24, 16, 32
    K, V, hid = _rand_bits(rng, (B, H, N, d)), _rand_bits(rng, (B, H, N, d)), _rand_bits(rng, (B, N, Dh))
    ho = torch.zeros((B, N, Dh), dtype=torch.bfloat16, device=DEV)
    Ko = torch.zeros((B, H, N, d), dtype=torch.bfloat16, device=DEV)
    Vo = torch.zeros((B, H, N, d), dtype=torch.bfloat16, device=DEV)
    olen = torch.zeros((B,), dtype=torch.int32, device=DEV)
    nkeep = torch.full((B,), -3, dtype=torch.int32, device=DEV)
    ws = vb.alloc_workspace(vb.OP_PRUNE_STEP, B=B, Nv=0)
    for budget in (0, 5):
        vb.vitcop_prune_step(vb.bf16_tensor(hid), vb.bf16_tensor(K), vb.bf16_tensor(V), 7, 0, 0, budget, ho, Ko, Vo,
                             olen, ws, n_keep_out=nkeep)
        assert vb.vitcop_poll_status(ws) == vb.OK
        assert np.all(olen.cpu().numpy() == N) and np.all(nkeep.cpu().numpy() == 0)
        assert np.array_equal(vb.bf16_bits(ho), hid) and np.array_equal(vb.bf16_bits(Ko), K)
        assert np.array_equal(vb.bf16_bits(Vo), V)


def test_paper_schedule_counts_through_the_chain():
    # Stage II -> III budgets of the paper's 88.9 % setting on m = 576: 172 tokens in, keep 77, then 15
    w = W.workload("c0")
    counts = [oracle.stage_count(576, p) for p in (0.3000, 0.1343, 0.0269)]
    assert counts == [172, 77, 15]
    import dataclasses
    w2 = dataclasses.replace(w, Nv=counts[0], budgets=(counts[1], counts[2]))
    _run_chain(w2)


# ======================================================================================= similarity / filter
@pytest.mark.parametrize("n,D,metric", [(1, 64, 0), (7, 64, 0), (129, 128, 0), (200, 128, 1), (577, 256, 0), (300, 1024, 1)])
def test_similarity_rows_small(n, D, metric):
    rng = np.random.default_rng(n)
    f = W.f32_to_bf16_bits(rng.standard_normal((2, n, D)).astype(np.float32) * (1 + 3 * rng.random((2, n, 1)).astype(np.float32)))
    r0, r1 = (0, n) if n < 200 else (n // 3, min(n, n // 3 + 150))
    got = gpu_similarity_rows(f, metric, r0, r1)
    for b in range(2):
        _, sim = oracle.feature_distance(f[b], metric, rows=(r0, r1), want_d2=False)
        if metric == 0:
            assert np.abs(got[b] - sim).max() <= SIM_ATOL
        else:
            x = W.bf16_bits_to_f32(f[b]).astype(np.float64)
            nrm = np.sqrt((x * x).sum(1))
            scale = nrm[r0:r1, None] * nrm[None, :]
            assert np.all(np.abs(got[b] - sim) <= GRAM_RTOL * scale)


@pytest.mark.parametrize("name,metric,tau", [("tiny", 0, 0.6), ("tiny", 1, 0.6), ("tiny", 0, -1.0), ("tiny", 0, 0.12), ("c0", 0, 0.6)])
def test_filter_small(name, metric, tau):
    w = W.workload(name)
    f = W.make_features(w)
    p = W.make_positions(w)
    d_c = w.d_c if metric == 0 else 8.0 * 4
    g = gpu_filter(f, p, metric, d_c, tau, w.n_centers)
    assert g.status == vb.OK
    assert np.all(g.n_clusters == w.n_centers)
    rep = []
    for b in range(f.shape[0]):
        check_vic_sample(f[b], p[b], metric, d_c, tau, w.n_centers, g.rho[b], g.delta2[b], g.parent[b], g.label[b], rep)
        assert len(np.unique(g.label[b])) == w.n_centers
    print("filter report", name, metric, tau, rep)


# Shapes of the one-kernel ("resident") sweep: one or two row blocks, a ragged last block, an odd and an even number
# of column blocks per row, and enough samples that every SM holds two units of work.
@pytest.mark.parametrize("B,n,metric,check", [(1, 129, 0, 1), (5, 300, 1, 2), (40, 257, 0, 3), (2, 1000, 0, 2),
                                              (3, 640, 0, 2)])
def test_filter_resident_shapes(B, n, metric, check):
    w = W.workload("tiny")
    f = W.make_features(w, n=n, B=B)
    p = np.tile(W.make_positions(w, n)[:1], (B, 1, 1))
    d_c = w.d_c if metric == 0 else 8.0 * 4
    nc = max(1, n // 20)
    g = gpu_filter(f, p, metric, d_c, w.tau, nc)
    assert g.status == vb.OK and np.all(g.n_clusters == nc)
    for b in sorted({0, B // 2, B - 1})[:check]:
        check_vic_sample(f[b], p[b], metric, d_c, w.tau, nc, g.rho[b], g.delta2[b], g.parent[b], g.label[b])


# Long samples (8192 tokens and more) keep the Gram tiles of the density sweep and run Eq. 3 as a separate pass over
# them: a ragged length (tiles that straddle the diagonal and the end of the sample), both metrics, with and
# without the spatial test.  Small feature width: the oracle's pairwise work stays cheap.
# With a radius, the tiles whose row block lies beyond it from their column blocks are neither kept nor read: 0.25 and
# 0.02 drop most of them (0.02: nearly all but the tiles on the diagonal).
@pytest.mark.parametrize("n,metric,tau", [(8200, 0, 0.6), (8321, 1, 0.6), (8200, 0, -1.0), (8192, 0, 0.25),
                                          (8250, 0, 0.02), (8200, 1, 0.25)])
def test_filter_long_sample_delta_pass(n, metric, tau):
    w = dataclasses.replace(W.workload("c4"), B=1, D=64, dup_rate=0.3)
    f = W.make_features(w, n=n, B=1)
    p = W.make_positions(w, n)[:1]
    d_c = w.d_c if metric == 0 else 40.0                 # (euclid: 1 % of the tokens have ten times the norm)
    nc = n // 20
    g = gpu_filter(f, p, metric, d_c, tau, nc)
    assert g.status == vb.OK and np.all(g.n_clusters == nc)
    rep = []
    check_vic_sample(f[0], p[0], metric, d_c, tau, nc, g.rho[0], g.delta2[0], g.parent[0], g.label[0], rep)
    print("filter long sample", n, metric, tau, rep)


def test_filter_long_samples_scattered_positions():
    """Two long samples in one call, one with positions in no order at all (no tile lies beyond the radius), one on the
    grid with a token whose position is not a number (it can be nobody's neighbour)."""
    n = 8192
    w = dataclasses.replace(W.workload("c4"), B=2, D=64, dup_rate=0.3)
    f = W.make_features(w, n=n, B=2)
    p = W.make_positions(w, n)[:2].copy()
    p[0] = np.random.default_rng(5).random((n, 2), dtype=np.float32)
    p[1, 4000] = np.nan
    nc = n // 20
    g = gpu_filter(f, p, 0, w.d_c, 0.3, nc)
    assert g.status == vb.OK and np.all(g.n_clusters == nc)
    for b in range(2):
        check_vic_sample(f[b], p[b], 0, w.d_c, 0.3, nc, g.rho[b], g.delta2[b], g.parent[b], g.label[b])


def test_filter_edge_cases():
    w = W.workload("tiny")
    # identical tokens: one cluster led by token 0
    f = np.tile(W.f32_to_bf16_bits(np.array([[1.0, 2.0, 3.0, 4.0] * 16], dtype=np.float32)), (1, 9, 1))
    g = gpu_filter(f, None, 0, 0.5, -1.0, 1)
    assert np.all(g.label == 0) and g.parent[0, 0] == -1 and np.all(g.parent[0, 1:] == 0)
    assert np.isinf(g.delta2[0, 0]) and np.all(g.delta2[0, 1:] <= 1e-6)
    assert np.allclose(g.rho, 8.0, rtol=1e-5)
    # n = 1 and n = 2
    f1 = W.make_features(w, n=1)
    g = gpu_filter(f1, W.make_positions(w, 1), 0, 0.5, 0.6, 1)
    assert np.all(g.label == 0) and np.all(g.rho == 0) and np.all(g.parent == -1)
    f2 = W.make_features(w, n=2)
    g = gpu_filter(f2, W.make_positions(w, 2), 0, 0.5, 0.6, 1)
    for b in range(f2.shape[0]):
        check_vic_sample(f2[b], W.make_positions(w, 2)[b], 0, 0.5, 0.6, 1, g.rho[b], g.delta2[b], g.parent[b], g.label[b])
    # tau = 0 with distinct positions: every token is an orphan; the non-centres adopt the nearest centre
    f = W.make_features(w, n=60)
    p = W.make_positions(w, 60)
    g = gpu_filter(f, p, 0, 0.5, 0.0, 5)
    assert np.all(g.parent == -1) and np.all(np.isinf(g.delta2))
    for b in range(f.shape[0]):
        check_vic_sample(f[b], p[b], 0, 0.5, 0.0, 5, g.rho[b], g.delta2[b], g.parent[b], g.label[b])
    # exact duplicates share a cluster; alpha path: ceil(200 * 0.05) = 10 centres
    f = W.make_features(w).copy()
    f[:, 31] = f[:, 30]
    g = gpu_filter(f, W.make_positions(w), 0, 0.5, 0.6, 0, alpha=0.05)
    assert np.all(g.n_clusters == 10) and np.all(g.label[:, 30] == g.label[:, 31])
    # every token a centre
    g = gpu_filter(f, W.make_positions(w), 0, 0.5, 0.6, 10 ** 6)
    assert np.array_equal(g.label, np.tile(np.arange(f.shape[1], dtype=np.int32), (f.shape[0], 1)))


def test_filter_then_quota_step_end_to_end():
    """Stage II as the paper runs it: VIC labels -> K-norm -> cluster quota -> compaction (tiny workload)."""
    w = W.workload("tiny")
    f = W.make_features(w)
    p = W.make_positions(w)
    g = gpu_filter(f, p, 0, w.d_c, w.tau, w.n_centers)
    stats = _run_chain(w, use_labels=g.label)
    assert stats["steps"] == len(w.budgets)


# ======================================================================================= Stage II in one call
# "tiny-wide": six samples of 203 tokens (ragged last chunk of eight), 3 heads of 256 -- a shape whose K-norm the
# one-kernel sweep takes in part (two 16-byte piece rounds per row), with the rest in the stand-alone kernel.
@pytest.mark.parametrize("name", ["tiny", "tiny-wide", "c0", "c1", "c2"])
def test_collaborative_step_equals_filter_then_prune_step(name):
    """vitcop_collaborative_step may reorder its kernels (the K-norm runs beside the clustering) but must return
    exactly what vitcop_redundancy_filter followed by vitcop_prune_step returns; that pair is checked against the
    oracle by the tests above."""
    if name == "tiny-wide":
        w = dataclasses.replace(W.workload("tiny"), B=6, Nv=203, H=3, d=256)
    else:
        w = W.workload(name)
    B, n = w.B, w.Nv
    feat, pos = vb.bf16_tensor(W.make_features(w)), torch.from_numpy(W.make_positions(w).copy()).to(DEV)
    K_b, V_b = W.make_kv(w, 0, n)
    tK, tV, th = vb.bf16_tensor(K_b), vb.bf16_tensor(V_b), vb.bf16_tensor(W.make_hidden(w))
    budget = w.budgets[0]
    Ncap = w.T + budget

    def outputs():
        z = lambda *s, dt: torch.zeros(s, dtype=dt, device=DEV)
        return dict(ho=z(B, Ncap, w.Dh, dt=torch.bfloat16), Ko=z(B, w.H, Ncap, w.d, dt=torch.bfloat16),
                    Vo=z(B, w.H, Ncap, w.d, dt=torch.bfloat16), olen=z(B, dt=torch.int32),
                    kpos=z(B, Ncap, dt=torch.int32), score=z(B, n, dt=torch.float32), kidx=z(B, n, dt=torch.int32),
                    nkeep=z(B, dt=torch.int32), label=z(B, n, dt=torch.int32), ncl=z(B, dt=torch.int32))

    ref = outputs()
    ws_f = vb.alloc_workspace(vb.OP_FILTER, B=B, Nv=n, D=w.D)
    ws_s = vb.alloc_workspace(vb.OP_PRUNE_STEP, B=B, Nv=n)
    vb.vitcop_redundancy_filter(feat, pos, ref["label"], ref["ncl"], ws_f, metric=0, d_c=w.d_c, tau=w.tau,
                                n_centers=w.n_centers)
    vb.vitcop_prune_step(th, tK, tV, w.vis_start, n, n, budget, ref["ho"], ref["Ko"], ref["Vo"], ref["olen"], ws_s,
                         label=ref["label"], kept_pos=ref["kpos"], score_out=ref["score"], keep_idx_out=ref["kidx"],
                         n_keep_out=ref["nkeep"])
    assert vb.vitcop_poll_status(ws_f) == vb.OK and vb.vitcop_poll_status(ws_s) == vb.OK
    for rep in range(2):                                   # twice: the second call runs on a used workspace
        got = outputs()
        ws = vb.alloc_workspace(vb.OP_COLLAB_STEP, B=B, Nv=n, D=w.D) if rep == 0 else ws
        vb.vitcop_collaborative_step(feat, pos, th, tK, tV, w.vis_start, budget, got["ho"], got["Ko"], got["Vo"],
                                     got["olen"], got["label"], got["ncl"], ws, metric=0, d_c=w.d_c, tau=w.tau,
                                     n_centers=w.n_centers, kept_pos=got["kpos"], score_out=got["score"],
                                     keep_idx_out=got["kidx"], n_keep_out=got["nkeep"])
        assert vb.vitcop_poll_status(ws) == vb.OK
        nk = ref["nkeep"].cpu().numpy()
        assert nk.min() > 0
        for key in ("label", "ncl", "score", "nkeep", "olen", "kpos"):
            assert torch.equal(got[key], ref[key]), key
        for b in range(B):
            assert torch.equal(got["kidx"][b, : nk[b]], ref["kidx"][b, : nk[b]])
        for key in ("ho", "Ko", "Vo"):
            assert torch.equal(got[key].view(torch.int16), ref[key].view(torch.int16)), key


def test_collaborative_step_replays_from_a_cuda_graph():
    """The one-call step only enqueues work on the caller's stream (one memset, cooperative and programmatically
    dependent launches): it can be captured once and replayed, with the same results as direct calls."""
    w = W.workload("c0")
    B, n = 2, w.Nv
    feat = vb.bf16_tensor(W.make_features(w, B=B))
    pos = torch.from_numpy(np.tile(W.make_positions(w), (B, 1, 1)).copy()).to(DEV)
    K_b, V_b = W.make_kv(w, 0, n, B=B)
    tK, tV = vb.bf16_tensor(K_b), vb.bf16_tensor(V_b)
    th = vb.bf16_tensor(W.make_hidden(w, B=B))
    budget, Ncap = w.budgets[-1], w.T + w.budgets[-1]
    z = lambda *s, dt: torch.zeros(s, dtype=dt, device=DEV)

    def outputs():
        return dict(ho=z(B, Ncap, w.Dh, dt=torch.bfloat16), Ko=z(B, w.H, Ncap, w.d, dt=torch.bfloat16),
                    Vo=z(B, w.H, Ncap, w.d, dt=torch.bfloat16), olen=z(B, dt=torch.int32),
                    label=z(B, n, dt=torch.int32), ncl=z(B, dt=torch.int32))

    def step(o, ws):
        vb.vitcop_collaborative_step(feat, pos, th, tK, tV, w.vis_start, budget, o["ho"], o["Ko"], o["Vo"], o["olen"],
                                     o["label"], o["ncl"], ws, metric=0, d_c=w.d_c, tau=w.tau, n_centers=w.n_centers)

    ref, ws_ref = outputs(), vb.alloc_workspace(vb.OP_COLLAB_STEP, B=B, Nv=n, D=w.D)
    step(ref, ws_ref)
    torch.cuda.synchronize()
    got, ws = outputs(), vb.alloc_workspace(vb.OP_COLLAB_STEP, B=B, Nv=n, D=w.D)
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    with torch.cuda.stream(side):
        step(got, ws)                                     # warm-up outside the capture (function attributes, maps)
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=side):
            step(got, ws)
    for _ in range(2):
        for t in got.values():
            t.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert vb.vitcop_poll_status(ws) == vb.OK
        assert int(ref["olen"].min()) > w.T
        for key in ("olen", "label", "ncl"):
            assert torch.equal(got[key], ref[key]), key
        for key in ("ho", "Ko", "Vo"):
            assert torch.equal(got[key].view(torch.int16), ref[key].view(torch.int16)), key
