"""The workspace-free variant of the fused pruning step, through the C ABI (``-m gpu``).

``vitcop_prune_step_static`` serves callers that cannot allocate device memory where they call it (no
allocator in reach, or one they must not touch mid-loop): its scratch is a buffer built into the library.
The buffer is shared by every call and keeps the previous call's contents, so this test makes two different
calls in a row and checks each against ``vitcop_prune_step`` with an ordinary workspace: same scores (within
the K-norm tolerance the other tests use; it is the same kernel, so in practice the same bits), same kept
indices, counts, positions and bit-identical compacted rows.  It also checks that a problem beyond the
built-in size is refused.  The file name sorts last so that a run stopping at the first failure has already
run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2601_17818_b200 import binding as vb
from paper_2601_17818_b200 import workloads as W

pytestmark = pytest.mark.gpu

KNORM_RTOL = 1e-5
DEV = "cuda"


def _outputs(B, H, Ncap, d, Dh, n):
    z = lambda *s, dt: torch.full(s, 0, dtype=dt, device=DEV)
    return dict(ho=z(B, Ncap, Dh, dt=torch.bfloat16), Ko=z(B, H, Ncap, d, dt=torch.bfloat16),
                Vo=z(B, H, Ncap, d, dt=torch.bfloat16), olen=z(B, dt=torch.int32), kpos=z(B, Ncap, dt=torch.int32),
                score=z(B, n, dt=torch.float32), kidx=z(B, n, dt=torch.int32), nkeep=z(B, dt=torch.int32))


def _both(w, step, n_vis, budget, label, own_buffers):
    """One problem through vitcop_prune_step (ordinary workspace) and through vitcop_prune_step_static.

    own_buffers=False leaves score / keep list / counts to the call: the static variant then keeps them in its
    built-in scratch, which is the memory this test is about."""
    K, V = W.make_kv(w, step, n_vis)
    hid = W.make_hidden(w)[:, : w.T + n_vis]
    tK, tV, th = vb.bf16_tensor(K), vb.bf16_tensor(V), vb.bf16_tensor(np.ascontiguousarray(hid))
    lab = None if label is None else torch.from_numpy(label).to(DEV)
    Ncap = w.T + min(budget, n_vis)
    ref = _outputs(w.B, w.H, Ncap, w.d, w.Dh, n_vis)
    ws = vb.alloc_workspace(vb.OP_PRUNE_STEP, B=w.B, Nv=n_vis)
    vb.vitcop_prune_step(th, tK, tV, w.vis_start, n_vis, n_vis, budget, ref["ho"], ref["Ko"], ref["Vo"], ref["olen"],
                         ws, label=lab, kept_pos=ref["kpos"], score_out=ref["score"], keep_idx_out=ref["kidx"],
                         n_keep_out=ref["nkeep"])
    assert vb.vitcop_poll_status(ws) == vb.OK
    got = _outputs(w.B, w.H, Ncap, w.d, w.Dh, n_vis)
    own = dict(score_out=got["score"], keep_idx_out=got["kidx"], n_keep_out=got["nkeep"]) if own_buffers else {}
    torch.cuda.synchronize()
    held, free = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
    vb.vitcop_prune_step_static(th, tK, tV, w.vis_start, n_vis, n_vis, budget, got["ho"], got["Ko"], got["Vo"],
                                got["olen"], label=lab, kept_pos=got["kpos"], **own)
    torch.cuda.synchronize()
    grown = (torch.cuda.memory_allocated() - held, free - torch.cuda.mem_get_info()[0])
    nk = ref["nkeep"].cpu().numpy()
    assert nk.max() > 0
    assert np.array_equal(got["olen"].cpu().numpy(), ref["olen"].cpu().numpy())
    assert np.array_equal(ref["olen"].cpu().numpy(), w.T + nk)
    if own_buffers:
        r_score, g_score = ref["score"].cpu().numpy(), got["score"].cpu().numpy()
        assert np.all(np.abs(g_score - r_score) <= KNORM_RTOL * np.abs(r_score))
        assert np.array_equal(got["nkeep"].cpu().numpy(), nk)
        for b in range(w.B):
            assert np.array_equal(got["kidx"].cpu().numpy()[b, : nk[b]], ref["kidx"].cpu().numpy()[b, : nk[b]])
    assert torch.equal(got["kpos"], ref["kpos"])
    for name in ("ho", "Ko", "Vo"):
        assert torch.equal(got[name].view(torch.int16), ref[name].view(torch.int16)), name
    return grown


def test_prune_step_static_matches_prune_step_twice_in_a_row():
    w = W.workload("tiny")
    labels = W.make_labels(5, w.B, w.Nv, w.n_centers)
    _both(w, 0, w.Nv, w.budgets[0], labels, own_buffers=True)    # first call: quota mode, full span
    # second call: plain mode, other (smaller) sizes, scores / keep list / counts in the built-in scratch, which
    # still holds what the larger first call left there
    _both(w, 1, 77, 13, None, own_buffers=False)
    # third: quota mode again on the scratch, over the plain call's leftovers
    grown = _both(w, 2, w.Nv, w.budgets[1], labels, own_buffers=False)
    # the call itself obtains no device memory, neither from torch's allocator nor from the driver (looked at
    # around the third call: every kernel it launches had been loaded by then)
    assert grown == (0, 0)


def test_prune_step_static_uses_the_whole_scratch_near_its_limit():
    """B * Nv_cap just below the limit: the keep list and the counts sit at the far end of the 4 MiB array."""
    import dataclasses
    w = dataclasses.replace(W.workload("tiny"), B=32, Nv=16256, T=8, H=1, d=8, Dh=8, budgets=(300, 100))
    need = vb.vitcop_workspace_bytes(vb.OP_PRUNE_STEP, B=w.B, Nv=w.Nv)
    assert (4 << 20) - 64 * 1024 < need <= (4 << 20)
    _both(w, 0, w.Nv, 300, None, own_buffers=False)
    labels = W.make_labels(9, w.B, w.Nv, 40)
    _both(w, 1, w.Nv, 500, labels, own_buffers=False)


def test_prune_step_static_refuses_oversized_problems():
    # B * Nv_cap * 8 bytes of scratch would exceed the built-in 4 MiB: rejected on the host, nothing launched
    B, H, N, d, Nv = 64, 1, 16384, 8, 16384
    K = torch.zeros((B, H, N, d), dtype=torch.bfloat16, device=DEV)
    Ko = torch.zeros((B, H, 8, d), dtype=torch.bfloat16, device=DEV)
    olen = torch.zeros((B,), dtype=torch.int32, device=DEV)
    assert vb.vitcop_workspace_bytes(vb.OP_PRUNE_STEP, B=B, Nv=Nv) > (4 << 20)
    with pytest.raises(vb.VitcopError) as e:
        vb.vitcop_prune_step_static(None, K, None, 0, Nv, Nv, 8, None, Ko, None, olen)
    assert e.value.status == vb.ERR_UNSUPPORTED
