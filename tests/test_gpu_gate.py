"""GPU parity: ec_entropy_gate (through the C ABI) against the fp64 oracle (Eq. 1,
Algorithm 1).  Tolerances: argmax and decisions bit-exact (decisions except where
|E - tau| < 1e-4), entropy within 1e-4 nats, confidence within 1e-5 relative."""
import math

import numpy as np
import pytest
import torch

import ec_synth as syn
import oracle
from _util import to_dev

pytestmark = pytest.mark.gpu

ENT_TOL = 1e-4


def _run_gpu(st, dtype, vocab, flags, tau, rows_per_seq, **kw):
    import paper_2603_18489_b200 as ec

    logits = to_dev(st)
    r = ec.ec_entropy_gate(logits, vocab, rows_per_seq, to_dev(flags), tau, **kw)
    torch.cuda.synchronize()
    return {k: (v.cpu().numpy() if v is not None else None) for k, v in r.items()}


def _compare(g, o, tau):
    assert np.array_equal(g["argmax"], o["argmax"])
    assert np.abs(g["entropy"].astype(np.float64) - o["entropy"]).max() <= ENT_TOL
    assert (np.abs(g["conf"].astype(np.float64) - o["conf"]) <= 1e-5 * o["conf"] + 1e-12).all()
    fin = np.isfinite(o["max_entropy"])
    assert np.array_equal(np.isfinite(g["max_entropy"]), fin)
    assert np.abs(g["max_entropy"][fin].astype(np.float64) - o["max_entropy"][fin]).max(initial=0) <= ENT_TOL
    band = np.abs(o["max_entropy"] - tau) < ENT_TOL
    assert np.array_equal(g["decision"][~band], o["decision"][~band])


@pytest.mark.parametrize("name,R,rps", [("c1_tiny_fp32", 32, 32), ("c2_llada_l768", 32, 32),
                                        ("c3_dream_l768", 32, 32), ("c5_llada_l4096_b8", 256, 32)])
def test_gate_on_benchmark_shapes(name, R, rps):
    w = syn.WORKLOADS[name]
    d = syn.logits_rows(R, w.vocab, w.dtype, cfg_id=w.cfg_id)
    flags = syn.decoded_flags(R, 16, rps, cfg_id=w.cfg_id)
    o = oracle.entropy_gate(d["logits"], w.dtype, w.vocab, flags, 1.5, rps)
    tau_med = float(np.float32(np.median(o["entropy"])))       # config-1 policy: tau = median row entropy
    for tau in (1.5, tau_med):
        o = oracle.entropy_gate(d["logits"], w.dtype, w.vocab, flags, tau, rps)
        g = _run_gpu(d["logits"], w.dtype, w.vocab, flags, tau, rps)
        _compare(g, o, tau)


@pytest.mark.parametrize("dtype", [syn.F32, syn.BF16])
@pytest.mark.parametrize("V,stride", [(1000, 1000), (1027, 1032), (2048, 2048), (2049, 2056), (5, 8),
                                      (8200, 8200), (40001, 40008)])
def test_gate_ragged_vocab_and_padded_rows(dtype, V, stride):
    R = 12
    d = syn.logits_rows(R, V, dtype, cfg_id=50 + V % 7, row_stride=stride)
    flags = syn.decoded_flags(R, 2, 4, cfg_id=51)
    o = oracle.entropy_gate(d["logits"], dtype, V, flags, 2.0, 4)
    g = _run_gpu(d["logits"], dtype, V, flags, 2.0, 4)
    _compare(g, o, 2.0)


@pytest.mark.parametrize("dtype", [syn.F32, syn.BF16])
def test_gate_closed_form_rows(dtype):
    V = 126464
    x = np.zeros((8, V), np.float32)
    x[1, :] = -3.25                           # uniform, shifted
    x[2, :] = -np.inf; x[2, V - 1] = 4.0      # one-hot at the very last column
    x[3, :] = -np.inf; x[3, [77, 90001]] = 1.0  # two-way tie: ln 2, argmax 77
    x[4, 5] = 12.25                           # spike
    x[5, :] = -3.0e38; x[5, 40000] = 0.0      # "finfo.min"-style masking
    x[6, V // 2:] = 8.0                       # half high, half low; ties -> first of the high half
    x[7, :16] = 8.0
    st = syn.encode(x, dtype)
    flags = np.ones(8, np.uint8)
    o = oracle.entropy_gate(st, dtype, V, flags, 1.5, 8)
    g = _run_gpu(st, dtype, V, flags, 1.5, 8)
    _compare(g, o, 1.5)
    H = g["entropy"]
    assert abs(H[0] - math.log(V)) < ENT_TOL and abs(H[1] - math.log(V)) < ENT_TOL
    assert H[2] == 0.0 and g["conf"][2] == 1.0 and g["argmax"][2] == V - 1
    assert abs(H[3] - math.log(2)) < 1e-6 and g["argmax"][3] == 77
    assert H[5] == 0.0 and g["argmax"][5] == 40000
    assert g["argmax"][6] == V // 2 and g["argmax"][0] == 0


def test_gate_flips_exactly_at_tau_and_ignores_unflagged_rows():
    V = 4096
    x = np.zeros((4, V), np.float32)           # rows 0, 2, 3 uniform: H = ln 4096
    x[1, :] = -np.inf; x[1, [3, 9]] = 0.0      # H = ln 2
    st = syn.encode(x, syn.F32)
    flags = np.array([0, 1, 0, 0], np.uint8)
    g0 = _run_gpu(st, syn.F32, V, flags, 1.5, 4)
    E = np.float32(g0["max_entropy"][0])       # the device's own fp32 E
    assert abs(float(E) - math.log(2)) < 1e-6
    assert g0["decision"][0] == 0              # unflagged high-entropy rows do not count
    g = _run_gpu(st, syn.F32, V, flags, float(E), 4)
    assert g["decision"][0] == 0               # E == tau -> skip
    g = _run_gpu(st, syn.F32, V, flags, float(np.nextafter(E, np.float32(-np.inf))), 4)
    assert g["decision"][0] == 1               # E > tau -> recompute
    flags[:] = 0
    g = _run_gpu(st, syn.F32, V, flags, -5.0, 4)
    assert g["max_entropy"][0] == -np.inf and g["decision"][0] == 0


def test_gate_optional_outputs_and_workspace_reuse():
    import paper_2603_18489_b200 as ec

    w = syn.C2
    d = syn.logits_rows(64, w.vocab, w.dtype, cfg_id=60)
    flags = syn.decoded_flags(64, 5, 16, cfg_id=60)
    o = oracle.entropy_gate(d["logits"], w.dtype, w.vocab, flags, 3.0, 16)
    logits, fl = to_dev(d["logits"]), to_dev(flags)
    ws = ec.new_workspace(ec.ec_entropy_gate_workspace_bytes(64, w.vocab))
    for _ in range(3):   # the same workspace serves consecutive calls without re-zeroing
        r = ec.ec_entropy_gate(logits, w.vocab, 16, fl, 3.0, workspace=ws, want_rows=False)
        torch.cuda.synchronize()
        assert r["argmax"] is None and r["entropy"] is None
        assert np.abs(r["max_entropy"].cpu().numpy() - o["max_entropy"]).max() <= ENT_TOL
        band = np.abs(o["max_entropy"] - 3.0) < ENT_TOL
        assert np.array_equal(r["decision"].cpu().numpy()[~band], o["decision"][~band])
    assert int(ws[: 64 * 8].to(torch.int32).sum()) == 0     # tickets are back to zero


def test_gate_shift_invariance_on_device():
    """H(x + c) = H(x): a property that holds at any size (checked on the device path alone)."""
    w = syn.C2
    d = syn.logits_rows(32, w.vocab, syn.F32, cfg_id=61)
    flags = np.ones(32, np.uint8)
    a = _run_gpu(d["logits"], syn.F32, w.vocab, flags, 1.5, 32)
    b = _run_gpu(d["logits"] + np.float32(16.0), syn.F32, w.vocab, flags, 1.5, 32)
    assert np.abs(a["entropy"] - b["entropy"]).max() < 5e-5


@pytest.mark.parametrize("name,R,rps", [("c1_tiny_fp32", 32, 32), ("c2_llada_l768", 32, 32), ("c5_llada_l4096_b8", 256, 32),
                                        ("c1_tiny_fp32", 15, 5), ("c3_dream_l768", 128, 64)])
def test_the_three_candidate_metrics(name, R, rps):
    """Section 5.3: max entropy, entropy sum and max confidence over the decoded rows, per sequence; empty decoded sets
    included (one sequence gets no flags).  Sum: within 1e-4 nats per decoded row; confidence: 1e-5 relative."""
    import paper_2603_18489_b200 as ec

    w = syn.WORKLOADS[name]
    d = syn.logits_rows(R, w.vocab, w.dtype, cfg_id=w.cfg_id, salt=3)
    flags = syn.decoded_flags(R, max(1, rps // 3), rps, cfg_id=w.cfg_id)
    flags[:rps] = 0                                                   # the first sequence decodes nothing
    o = oracle.entropy_gate(d["logits"], w.dtype, w.vocab, flags, 1.5, rps)
    m = oracle.gate_metrics(o["entropy"], o["conf"], flags, rps)
    g = ec.ec_entropy_gate_metrics(to_dev(d["logits"]), w.vocab, rps, to_dev(flags), 1.5)
    torch.cuda.synchronize()
    g = {k: v.cpu().numpy() for k, v in g.items()}
    _compare(g, o, 1.5)
    n_dec = flags.reshape(-1, rps).sum(axis=1)
    assert np.all(np.abs(g["entropy_sum"].astype(np.float64) - m["entropy_sum"]) <= ENT_TOL * np.maximum(n_dec, 1))
    fin = np.isfinite(m["max_conf"])
    assert np.array_equal(np.isfinite(g["max_conf"]), fin) and not fin[0] and g["entropy_sum"][0] == 0.0
    assert np.all(np.abs(g["max_conf"][fin].astype(np.float64) - m["max_conf"][fin]) <= 1e-5 * m["max_conf"][fin])


@pytest.mark.parametrize("dtype,R,V,stride,rps", [(syn.F32, 96, 126464, 126464, 32), (syn.BF16, 200, 126466, 126472, 40),
                                                  (syn.F32, 48, 152064, 152064, 48)])
def test_gate_on_inputs_large_enough_for_the_per_thread_loads(dtype, R, V, stride, rps):
    """From 24 MB of logits on, the gate's threads load their own vectors (rolling registers) instead of reading a
    bulk-copy ring: both storage types, a padded stride with a ragged vocabulary, sequences of 40 and 48 rows (the
    benchmark shape [256, 126464] bf16 is covered by test_gate_on_benchmark_shapes)."""
    assert R * V * (4 if dtype == syn.F32 else 2) >= 24 << 20
    st = syn.logits_rows(R, V, dtype, cfg_id=8, row_stride=stride)
    flags = syn.decoded_flags(R, 7, rps, cfg_id=8)
    tau = 2.0
    g = _run_gpu(st["logits"], dtype, V, flags, tau, rps)
    o = oracle.entropy_gate(st["logits"], dtype, V, flags, tau, rps)
    _compare(g, o, tau)
