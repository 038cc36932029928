"""GPU parity: ec_kv_refresh against the oracle, byte for byte (Section 4.2)."""
import numpy as np
import pytest
import torch

import ec_synth as syn
import oracle
from _util import to_dev, to_storage

pytestmark = pytest.mark.gpu


def _case(w, n_active, idx):
    import paper_2603_18489_b200 as ec

    t = syn.attn_inputs(w, n_active, active_idx=idx)
    idx = t["active_idx"]
    kc, vc = t["k_cache"].copy(), t["v_cache"].copy()
    oracle.kv_refresh(kc, vc, t["k_new"], t["v_new"], idx, w.dtype)
    d = ec.make_desc(w.batch, w.ctx_len, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype)
    gk, gv = to_dev(t["k_cache"]), to_dev(t["v_cache"])
    ec.ec_kv_refresh(d, gk, gv, to_dev(t["k_new"]), to_dev(t["v_new"]), to_dev(idx))
    torch.cuda.synchronize()
    assert np.array_equal(to_storage(gk), kc)
    assert np.array_equal(to_storage(gv), vc)


@pytest.mark.parametrize("name", ["c1_tiny_fp32", "c2_llada_l768", "c3_dream_l768", "c4_llada_l2048"])
def test_refresh_skip_and_recompute_rows(name):
    w = syn.WORKLOADS[name]
    _case(w, w.n_skip_rows, None)
    _case(w, w.ctx_len, None)


def test_refresh_batched_random_rows_and_empty():
    import paper_2603_18489_b200 as ec

    w = syn.Workload(92, "r", syn.BF16, 3, 8, 2, 128, 100, 57, 32, 2, 64)
    idx = syn.arbitrary_active_idx(3, w.ctx_len, 41, seed=8)
    _case(w, 41, idx)
    w32 = syn.Workload(93, "r", syn.F32, 2, 4, 4, 64, 10, 23, 4, 0, 64)
    _case(w32, 33, syn.arbitrary_active_idx(2, 33, 33, seed=9))   # every row, permuted
    d = ec.make_desc(1, 16, 2, 2, 64, ec.EC_F32)
    z = torch.zeros(1, 2, 16, 64, device="cuda")
    e = torch.zeros(1, 0, 2, 64, device="cuda")
    ec.ec_kv_refresh(d, z, z, e, e, torch.zeros(1, 0, dtype=torch.int32, device="cuda"))   # n_active == 0: no-op


def test_refresh_skips_out_of_range_indices():
    import paper_2603_18489_b200 as ec

    w = syn.Workload(94, "r", syn.BF16, 1, 2, 2, 64, 8, 8, 4, 0, 64)
    t = syn.attn_inputs(w, 4, k_recent=0)
    idx = np.array([[3, -1, 16, 7]], np.int32)        # two indices outside [0, 16)
    gk, gv = to_dev(t["k_cache"]), to_dev(t["v_cache"])
    d = ec.make_desc(1, 16, 2, 2, 64, ec.EC_BF16)
    ec.ec_kv_refresh(d, gk, gv, to_dev(t["k_new"]), to_dev(t["v_new"]), to_dev(idx))
    torch.cuda.synchronize()
    kc = t["k_cache"].copy()
    kc[0, :, 3, :] = t["k_new"][0, 0]
    kc[0, :, 7, :] = t["k_new"][0, 3]
    assert np.array_equal(to_storage(gk), kc)
