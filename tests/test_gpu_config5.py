"""GPU parity at the full-depth benchmark configuration (LLaDA geometry, L = 4096, batch 1 and 8; Algorithm 1 and
Appendix A of the paper): the skip step and the recompute step of a whole batch, a step in which the sequences of
the batch took different decisions, the paper's default budget k = 64 at batch 8, and a 64-step replay over
several layers.  The oracle computes every row where that takes seconds and a seeded sample of query rows
otherwise (rows are independent, so the sampled rows are exact); refreshed caches are compared byte for byte.
Each test also names the kernel the dispatch picks for its shape, so the parity result is tied to that kernel."""
import functools

import numpy as np
import pytest
import torch

import ec_synth as syn
import oracle
from _replay import ReplayState, decoded_this_step, step_inputs
from _util import to_dev, to_f64, to_storage

pytestmark = pytest.mark.gpu

BF16_TOL = 1e-2


def _sample_rows(n, count, seed):
    if n <= count:
        return list(range(n))
    r = np.random.Generator(np.random.PCG64(seed)).choice(n, count - 2, replace=False).tolist()
    return sorted(set(r + [0, n - 1]))


@functools.lru_cache(maxsize=1)
def _batch8_full():
    """Seeded tensors of the batch-8 configuration: caches plus fresh q / k / v for every row."""
    return syn.attn_inputs(syn.C5B8, syn.C5B8.ctx_len)


def _rows_inputs(w, n, seed, idx):
    """q / k_new / v_new for n active rows (benchmark law N(0,1)/sqrt(D)); the caches come from _batch8_full()."""
    rng = np.random.Generator(np.random.PCG64(seed))
    std = np.float32(1.0 / np.sqrt(w.head_dim))
    draw = lambda h: syn.encode(rng.standard_normal((w.batch, n, h, w.head_dim), dtype=np.float32) * std, w.dtype)
    return dict(q=draw(w.n_q_heads), k_new=draw(w.n_kv_heads), v_new=draw(w.n_kv_heads), active_idx=idx)


def _run_and_compare(w, d_batch, q, kn, vn, kc_np, vc_np, idx, row_sel, expect_kernel):
    """One ec_attend call on `d_batch` sequences against the oracle; returns the refreshed caches (numpy)."""
    import paper_2603_18489_b200 as ec

    n = q.shape[1]
    d = ec.make_desc(d_batch, w.ctx_len, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype)
    name = ec.ec_attend_kernel_name(d, n, True, idx is not None)
    assert name.startswith(expect_kernel), name
    gk, gv = to_dev(kc_np), to_dev(vc_np)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = ec.ec_attend(d, to_dev(q), to_dev(kn), to_dev(vn), gk, gv, to_dev(idx), dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    okc, ovc = kc_np.copy(), vc_np.copy()
    ref = oracle.refresh_and_attend(q, kn, vn, okc, ovc, idx, w.dtype, row_sel=row_sel)
    got = to_f64(out if row_sel is None else out[:, row_sel])
    err = np.abs(got - ref).max()
    assert err <= BF16_TOL, err
    assert np.array_equal(to_storage(gk), okc) and np.array_equal(to_storage(gv), ovc)
    return okc, ovc


def test_batch8_skip_step_every_row():
    """The batch-8 skip step of the benchmark (8 x 32 heads, 34 rows over 4096 keys): rows on the M axis, one CTA
    per (sequence, head), 64 key tiles through the three-stage ring."""
    w = syn.C5B8
    t = _batch8_full()
    idx = syn.active_rows(w, block_no=7, shuffle=True)
    r = _rows_inputs(w, w.n_skip_rows, 501, idx)
    _run_and_compare(w, w.batch, r["q"], r["k_new"], r["v_new"], t["k_cache"], t["v_cache"], idx, None,
                     "attend_skip_kernel<1> grid=(1,256) cluster=1")


@pytest.mark.parametrize("n,kernel", [(96, "attend_skip_kernel<1> grid=(1,256)"), (160, "attend_skip_kernel<2> grid=(1,256)"),
                                      (200, "attend_skip_kernel<2> grid=(1,256)")])
def test_batch8_skip_step_with_the_papers_budgets(n, kernel):
    """k = 64 (the paper's default: 96 rows) and two points of its grid at batch 8, rows scattered over the context;
    the oracle computes 20 sampled rows per sequence."""
    w = syn.C5B8
    t = _batch8_full()
    idx = syn.arbitrary_active_idx(w.batch, w.ctx_len, n, seed=900 + n)
    r = _rows_inputs(w, n, 600 + n, idx)
    _run_and_compare(w, w.batch, r["q"], r["k_new"], r["v_new"], t["k_cache"], t["v_cache"], idx,
                     _sample_rows(n, 20, n), kernel)


def test_batch5_ragged_context_skip_step():
    """Five sequences at a context that is no multiple of the key tile (L = 700): more (sequence, head) pairs than
    one wave of clusters, so one CTA per pair streams all eleven 64-key tiles, the last one ragged."""
    w = syn.Workload(91, "b5_l700", syn.BF16, 5, 32, 32, 128, 444, 256, 32, 2, 64)
    idx = syn.arbitrary_active_idx(w.batch, w.ctx_len, 34, seed=17)
    t = syn.attn_inputs(w, 34, active_idx=idx)
    _run_and_compare(w, w.batch, t["q"], t["k_new"], t["v_new"], t["k_cache"], t["v_cache"], idx, None,
                     "attend_skip_kernel<1> grid=(1,160) cluster=1")
    # the same with a softmax that is far from uniform (score std 4) and a position list in the last, ragged tile
    idx2 = np.tile(np.arange(700 - 34, 700, dtype=np.int32), (w.batch, 1))
    t2 = syn.attn_inputs(w, 34, active_idx=idx2, std_qk=2.0 / np.sqrt(np.sqrt(128)), std_v=0.5, salt=1)
    _run_and_compare(w, w.batch, t2["q"], t2["k_new"], t2["v_new"], t2["k_cache"], t2["v_cache"], idx2, None,
                     "attend_skip_kernel<1>")


def test_batch8_recompute_step_sampled_rows():
    w = syn.C5B8
    t = _batch8_full()
    rows = _sample_rows(w.ctx_len, 18, 5)
    _run_and_compare(w, w.batch, t["q"], t["k_new"], t["v_new"], t["k_cache"], t["v_cache"], None, rows,
                     "attend_dense_kernel grid=(16,256)")


def test_step_with_mixed_decisions_across_the_batch():
    """Sequences {0, 1, 4} of the batch skip, the others recompute (per-sequence decisions of the gate): one call
    per run of consecutive sequences of a kind, on batch slices of the same tensors.  Outputs per sequence against
    the oracle, then the whole batch's caches byte for byte."""
    import paper_2603_18489_b200 as ec

    w = syn.C5B8
    t = _batch8_full()
    L = w.ctx_len
    skip_seqs = [0, 1, 4]
    rec_seqs = [b for b in range(w.batch) if b not in skip_seqs]
    idx = syn.active_rows(w, block_no=11)
    r = _rows_inputs(w, w.n_skip_rows, 777, idx)
    gk, gv = to_dev(t["k_cache"]), to_dev(t["v_cache"])
    gq_s, gkn_s, gvn_s, gidx = to_dev(r["q"]), to_dev(r["k_new"]), to_dev(r["v_new"]), to_dev(idx)
    gq_r, gkn_r, gvn_r = to_dev(t["q"]), to_dev(t["k_new"]), to_dev(t["v_new"])
    out_s, out_r = torch.zeros_like(gq_s), torch.zeros_like(gq_r)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    kinds = set()
    for b0, nb in syn.consecutive_runs(skip_seqs):
        d = ec.make_desc(nb, L, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype)
        kinds.add(ec.ec_attend_kernel_name(d, w.n_skip_rows, True, True).split(" ")[0])
        sl = slice(b0, b0 + nb)
        ec.ec_attend(d, gq_s[sl], gkn_s[sl], gvn_s[sl], gk[sl], gv[sl], gidx[sl], out=out_s[sl], dev_status=status)
    for b0, nb in syn.consecutive_runs(rec_seqs):
        d = ec.make_desc(nb, L, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype)
        kinds.add(ec.ec_attend_kernel_name(d, L, True, False).split(" ")[0])
        sl = slice(b0, b0 + nb)
        ec.ec_attend(d, gq_r[sl], gkn_r[sl], gvn_r[sl], gk[sl], gv[sl], None, out=out_r[sl], dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert kinds == {"attend_skip_keys_kernel<48>", "attend_dense_kernel"}
    okc, ovc = t["k_cache"].copy(), t["v_cache"].copy()
    rows = _sample_rows(L, 12, 9)
    for b in range(w.batch):
        sl = slice(b, b + 1)
        if b in skip_seqs:
            ref = oracle.refresh_and_attend(r["q"][sl], r["k_new"][sl], r["v_new"][sl], okc[sl], ovc[sl], idx[sl], w.dtype)
            got = to_f64(out_s[sl])
        else:
            ref = oracle.refresh_and_attend(t["q"][sl], t["k_new"][sl], t["v_new"][sl], okc[sl], ovc[sl], None, w.dtype,
                                            row_sel=rows)
            got = to_f64(out_r[sl][:, rows])
        assert np.abs(got - ref).max() <= BF16_TOL, b
    assert np.array_equal(to_storage(gk), okc) and np.array_equal(to_storage(gv), ovc)


def test_config5_sixty_four_step_replay_over_three_layers():
    """The fifth configuration's trace: 64 denoising steps at L = 4096 over three layers with distinct caches, the
    skip / recompute pattern driven by the gate on seeded logits whose sigma drifts from step to step.  Per step: the
    gate's maximum entropy (<= 1e-4 nats) and decision against the oracle (the oracle's decision drives both when
    |E - tau| < 1e-4), per layer the attention output on sampled query rows; at the end every layer's caches byte for
    byte.  The loop's bookkeeping (history, recent rows, skip_flag, dt) is the host harness's."""
    import paper_2603_18489_b200 as ec

    w = syn.C5
    n_layers, n_steps, k = 3, 64, w.k_recent
    centre = lambda s: syn.drifting_sigma_centre(s)
    # tau: the 85th percentile of the per-step maximum entropies (gate-only pre-pass of the oracle)
    st = ReplayState(w)
    E, all_flags, all_logits = [], [], []
    for s in range(n_steps):
        lg = syn.logits_rows(w.block, w.vocab, w.dtype, cfg_id=w.cfg_id, step=s, sigma_lo=max(0.25, centre(s) - 1.5),
                             sigma_hi=centre(s) + 1.5)["logits"]
        flags = decoded_this_step(st, s, 4)
        if not flags.any():
            st.block_start = min(st.block_start + w.block, w.ctx_len - w.block)
            st.masked[:] = True
            flags = decoded_this_step(st, s, 4)
        o = oracle.entropy_gate(lg, w.dtype, w.vocab, flags, 0.0, w.block)
        E.append(o["max_entropy"][0])
        all_flags.append(flags)
        all_logits.append(lg)
        st.record(flags, 0)
    tau = float(np.float32(np.quantile(E, 0.85)))

    d = ec.make_desc(1, w.ctx_len, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype)
    caches = [syn.attn_inputs(w, w.ctx_len, salt=10 + l) for l in range(n_layers)]
    okc = [c["k_cache"].copy() for c in caches]
    ovc = [c["v_cache"].copy() for c in caches]
    gk = [to_dev(c["k_cache"]) for c in caches]
    gv = [to_dev(c["v_cache"]) for c in caches]
    del caches
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    st = ReplayState(w)
    pattern = ""
    for s in range(n_steps):
        idx = st.active_rows(k)
        n_active = w.ctx_len if idx is None else idx.size
        pattern += "R" if idx is None else "s"
        idx_b = None if idx is None else idx[None, :].astype(np.int32)
        rows = _sample_rows(n_active, 10, 31 * s)
        for l in range(n_layers):
            rng = np.random.Generator(np.random.PCG64(40_000 + 100 * s + l))
            std = np.float32(1.0 / np.sqrt(w.head_dim))
            draw = lambda h: syn.encode(rng.standard_normal((1, n_active, h, w.head_dim), dtype=np.float32) * std, w.dtype)
            q, kn, vn = draw(w.n_q_heads), draw(w.n_kv_heads), draw(w.n_kv_heads)
            out = ec.ec_attend(d, to_dev(q), to_dev(kn), to_dev(vn), gk[l], gv[l], to_dev(idx_b), dev_status=status)
            ref = oracle.refresh_and_attend(q, kn, vn, okc[l], ovc[l], idx_b, w.dtype, row_sel=rows)
            assert np.abs(to_f64(out[:, rows]) - ref).max() <= BF16_TOL, (s, l)
        flags = decoded_this_step(st, s, 4)
        if not flags.any():            # block finished: open the next one, as the pre-pass did at this step
            st.block_start = min(st.block_start + w.block, w.ctx_len - w.block)
            st.masked[:] = True
            flags = decoded_this_step(st, s, 4)
        assert np.array_equal(flags, all_flags[s])
        o = oracle.entropy_gate(all_logits[s], w.dtype, w.vocab, flags, tau, w.block)
        g = ec.ec_entropy_gate(to_dev(all_logits[s]), w.vocab, w.block, to_dev(flags), tau)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert abs(float(g["max_entropy"][0]) - o["max_entropy"][0]) <= 1e-4, s
        if abs(o["max_entropy"][0] - tau) >= 1e-4:
            assert int(g["decision"][0]) == int(o["decision"][0]), s
        st.record(flags, int(o["decision"][0]))
    assert pattern[0] == "R" and 4 <= pattern.count("R") <= 24 and "s" in pattern, pattern
    for l in range(n_layers):
        assert np.array_equal(to_storage(gk[l]), okc[l]) and np.array_equal(to_storage(gv[l]), ovc[l]), l
