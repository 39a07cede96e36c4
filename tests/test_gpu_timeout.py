"""The give-up path of the Gram kernels' bounded waits, through the C ABI (``-m gpu``).

Every device-side wait of the library is bounded; when one runs out the CTA abandons its work, lets what it has in
flight finish, frees its tensor memory, and the call reports VITCOP_ERR_TIMEOUT through the status word.  No wait
runs out in normal operation, so these tests send one role of every CTA down that path (vitcop_set_wait_limit with
``expire_roles``) while the other roles have copies and tensor-core work in flight, and check that the call
returns, reports the timeout, and that the same workspace gives correct results on the next normal call.
"""
import numpy as np
import pytest
import torch

from paper_2601_17818_b200 import binding as vb
from paper_2601_17818_b200 import workloads as W

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from gpu_helpers import DEV

ROLE_LOAD, ROLE_MMA, ROLE_EPILOGUE = 1, 2, 4


@pytest.fixture(autouse=True)
def _restore_default_limit():
    yield
    vb.vitcop_set_wait_limit(0, 0)


def _filter_call(feat, pos, w, ws, out):
    vb.vitcop_redundancy_filter(feat, pos, out["label"], out["ncl"], ws, metric=0, d_c=w.d_c, tau=w.tau,
                                n_centers=out["nc"], rho=out["rho"], delta2=out["d2"], parent=out["par"])
    return vb.vitcop_poll_status(ws)


# B = 2 runs the one-kernel sweep (accumulators resident in tensor memory, cooperative launch, flags between CTAs);
# B = 80 exceeds what one wave of CTAs can keep resident and runs the diagonal / density / delta sweeps.
@pytest.mark.parametrize("B,n", [(2, 200), (80, 300)])
@pytest.mark.parametrize("roles", [ROLE_EPILOGUE, ROLE_MMA, ROLE_LOAD])
def test_filter_reports_timeout_and_recovers(B, n, roles):
    w = W.workload("tiny")
    f = W.make_features(w, n=n, B=B)
    feat = vb.bf16_tensor(f)
    pos = torch.from_numpy(np.tile(W.make_positions(w, n)[:1], (B, 1, 1)).copy()).to(DEV)
    nc = max(1, n // 20)

    def outputs():
        z = lambda *s, dt: torch.zeros(s, dtype=dt, device=DEV)
        return dict(label=z(B, n, dt=torch.int32), ncl=z(B, dt=torch.int32), rho=z(B, n, dt=torch.float32),
                    d2=z(B, n, dt=torch.float32), par=z(B, n, dt=torch.int32), nc=nc)

    ws = vb.alloc_workspace(vb.OP_FILTER, B=B, Nv=n, D=w.D)
    ref = outputs()
    assert _filter_call(feat, pos, w, ws, ref) == vb.OK
    vb.vitcop_set_wait_limit(0, roles)
    bad = outputs()
    assert _filter_call(feat, pos, w, ws, bad) == vb.ERR_TIMEOUT           # the call returned and says so
    vb.vitcop_set_wait_limit(0, 0)
    got = outputs()
    assert _filter_call(feat, pos, w, ws, got) == vb.OK                    # same workspace, next call is clean
    for key in ("label", "ncl", "rho", "d2", "par"):
        assert torch.equal(got[key], ref[key]), key


def test_similarity_rows_reports_timeout_and_recovers():
    w = W.workload("tiny")
    f = W.make_features(w)
    feat = vb.bf16_tensor(f)
    B, n, D = feat.shape
    ws = vb.alloc_workspace(vb.OP_SIMILARITY, B=B, Nv=n, D=D)
    ref = torch.zeros((B, n, n), dtype=torch.float32, device=DEV)
    vb.vitcop_similarity_rows(feat, 0, 0, n, ref, ws)
    assert vb.vitcop_poll_status(ws) == vb.OK
    vb.vitcop_set_wait_limit(0, ROLE_EPILOGUE)
    vb.vitcop_similarity_rows(feat, 0, 0, n, torch.zeros_like(ref), ws)
    assert vb.vitcop_poll_status(ws) == vb.ERR_TIMEOUT
    vb.vitcop_set_wait_limit(0, 0)
    got = torch.zeros_like(ref)
    vb.vitcop_similarity_rows(feat, 0, 0, n, got, ws)
    assert vb.vitcop_poll_status(ws) == vb.OK and torch.equal(got, ref)


def test_one_call_step_reports_timeout_and_recovers():
    """The one-kernel sweep with its K-norm side work (bulk copies streamed by the load and MMA warps)."""
    w = W.workload("tiny")
    B, n = w.B, w.Nv
    feat = vb.bf16_tensor(W.make_features(w))
    pos = torch.from_numpy(W.make_positions(w).copy()).to(DEV)
    K_b, V_b = W.make_kv(w, 0, n)
    tK, tV, th = vb.bf16_tensor(K_b), vb.bf16_tensor(V_b), vb.bf16_tensor(W.make_hidden(w))
    budget, Ncap = w.budgets[0], w.T + w.budgets[0]

    def run(ws):
        z = lambda *s, dt: torch.zeros(s, dtype=dt, device=DEV)
        o = dict(ho=z(B, Ncap, w.Dh, dt=torch.bfloat16), Ko=z(B, w.H, Ncap, w.d, dt=torch.bfloat16),
                 Vo=z(B, w.H, Ncap, w.d, dt=torch.bfloat16), olen=z(B, dt=torch.int32), label=z(B, n, dt=torch.int32),
                 ncl=z(B, dt=torch.int32), score=z(B, n, dt=torch.float32))
        vb.vitcop_collaborative_step(feat, pos, th, tK, tV, w.vis_start, budget, o["ho"], o["Ko"], o["Vo"], o["olen"],
                                     o["label"], o["ncl"], ws, metric=0, d_c=w.d_c, tau=w.tau, n_centers=w.n_centers,
                                     score_out=o["score"])
        return vb.vitcop_poll_status(ws), o

    ws = vb.alloc_workspace(vb.OP_COLLAB_STEP, B=B, Nv=n, D=w.D)
    st, ref = run(ws)
    assert st == vb.OK
    for roles in (ROLE_EPILOGUE, ROLE_MMA):
        vb.vitcop_set_wait_limit(0, roles)
        st, _ = run(ws)
        assert st == vb.ERR_TIMEOUT
        vb.vitcop_set_wait_limit(0, 0)
        st, got = run(ws)
        assert st == vb.OK
        for key in ("label", "olen", "score"):
            assert torch.equal(got[key], ref[key]), key
        for key in ("ho", "Ko", "Vo"):
            assert torch.equal(got[key].view(torch.int16), ref[key].view(torch.int16)), key
