"""The schedule exactly as bench.py runs it (one Stage II call, then Stage III calls fed by the lengths the previous
call left on the device), checked stage by stage against the oracle on the same seeded inputs (``-m gpu``)."""
import importlib.util
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2601_17818_b200 import binding as vb
from paper_2601_17818_b200 import workloads as W

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from gpu_helpers import KNORM_RTOL, oracle_band_check, oracle_quota_band_check

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench_module():
    spec = importlib.util.spec_from_file_location("bench_under_test", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


@pytest.mark.parametrize("name", ["c0", "c3", "c4"])
def test_benchmarked_schedule_matches_the_oracle(name):
    bench = _bench_module()
    w = W.workload(name)
    dev = torch.device("cuda", 0)
    host = bench.host_arrays(w)
    sc = bench.Schedule(w, torch, vb, dev)
    pinned = {k: (torch.from_numpy(v.view(np.int16)).view(torch.bfloat16) if v.dtype == np.uint16 else torch.from_numpy(v))
              for k, v in host.items()}
    sc.upload(pinned, non_blocking=False)
    sc.run()
    torch.cuda.synchronize()
    assert vb.vitcop_poll_status(sc.ws_c) == vb.OK
    g_label = sc.label.cpu().numpy()
    hidden = [host["hidden"][b] for b in range(w.B)]       # the oracle's own chain of hidden states
    n_vis = [w.Nv] * w.B
    for s, budget in enumerate(w.budgets):
        if s > 0:
            assert vb.vitcop_poll_status(sc.ws_s[s]) == vb.OK
        nk = sc.nkeep[s].cpu().numpy()
        olen = sc.olen[s].cpu().numpy()
        kpos = sc.kpos[s].cpu().numpy()
        g_ho, g_Ko, g_Vo = vb.bf16_bits(sc.ho[s]), vb.bf16_bits(sc.Ko[s]), vb.bf16_bits(sc.Vo[s])
        for b in range(w.B):
            N_b = w.T + n_vis[b]
            K = np.ascontiguousarray(host[f"K{s}"][b][:, :N_b])
            V = np.ascontiguousarray(host[f"V{s}"][b][:, :N_b])
            score = oracle.knorm(K[None], w.vis_start, n_vis[b])[0]
            keep = kpos[b, w.vis_start: w.vis_start + nk[b]] - w.vis_start
            if s == 0:
                oracle_quota_band_check(score, g_label[b], keep, budget, KNORM_RTOL)      # Eq. 5 with the step's own labels
            else:
                oracle_band_check(score, keep, budget, KNORM_RTOL)                        # plain top-k of Stage III
                assert nk[b] == min(budget, n_vis[b])
            o = oracle.compact(hidden[b][:N_b], K, V, N_b, w.vis_start, n_vis[b], keep, w.T + len(keep))
            L = o["out_len"]
            assert olen[b] == L == w.T + nk[b]
            assert np.array_equal(kpos[b, :L], o["kept_pos"][:L])
            assert np.array_equal(g_ho[b, :L], o["hidden"][:L])
            assert np.array_equal(g_Ko[b, :, :L], o["K"][:, :L]) and np.array_equal(g_Vo[b, :, :L], o["V"][:, :L])
            hidden[b] = o["hidden"][:L]
            n_vis[b] = int(nk[b])
    # the count bench.py turns into its metric
    assert w.B * w.Nv - int(sc.nkeep[-1].sum()) == sum(w.Nv - n for n in n_vis)
