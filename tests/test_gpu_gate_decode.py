"""GPU parity: ec_entropy_gate_decode (the gate with confidence-based parallel decoding in front of it) against
the oracle.  Row statistics as for the gate (argmax exact, entropy 1e-4 nats, confidence 1e-5 relative); the
decoded set, the updated mask and the token writes are integer work and must match exactly, except where a
confidence lies within 1e-5 relative of the threshold (or, when the single best row is taken, of the runner-up):
there both answers are valid and only validity is checked."""
import numpy as np
import pytest
import torch

import ec_synth as syn
import oracle
from _util import to_dev

pytestmark = pytest.mark.gpu


def _logits(R, V, dtype, seed, n_spiked, spike=14.0, stride=None, sigma_hi=8.0):
    """Gaussian rows (sigma in [0.5, 8]); `n_spiked` of them get one logit raised so that its probability is high."""
    d = syn.logits_rows(R, V, dtype, cfg_id=seed, row_stride=stride, sigma_hi=sigma_hi)
    x = syn.decode_f64(d["logits"], dtype)
    rng = np.random.Generator(np.random.PCG64(900 + seed))
    rows = rng.choice(R, size=min(n_spiked, R), replace=False)
    for r in rows:
        x[r, int(rng.integers(0, V))] += spike + float(rng.random()) * 6.0
    return syn.encode(x.astype(np.float32), dtype)


def _run(lg, dtype, V, masked, thr, tau, rps):
    import paper_2603_18489_b200 as ec

    m = to_dev(masked.copy())
    tok = torch.full((masked.size,), -7, dtype=torch.int32, device="cuda")
    r = ec.ec_entropy_gate_decode(to_dev(lg), V, rps, m, thr, tau, tok)
    torch.cuda.synchronize()
    out = {k: v.cpu().numpy() for k, v in r.items()}
    out["masked_next"], out["tokens"] = m.cpu().numpy(), tok.cpu().numpy()
    return out


def _check(lg, dtype, V, masked, thr, tau, rps):
    o = oracle.entropy_gate_decode(lg, dtype, V, masked, thr, tau, rps)
    g = _run(lg, dtype, V, masked, thr, tau, rps)
    assert np.array_equal(g["argmax"], o["argmax"])
    assert np.abs(g["entropy"].astype(np.float64) - o["entropy"]).max() <= 1e-4
    assert (np.abs(g["conf"].astype(np.float64) - o["conf"]) <= 1e-5 * o["conf"] + 1e-12).all()
    n_seq = masked.size // rps
    n_exact = 0
    for b in range(n_seq):
        sl = slice(b * rps, (b + 1) * rps)
        conf, m = o["conf"][sl], masked[sl].astype(bool)
        gd, od = g["decoded"][sl], o["decoded"][sl]
        near_thr = m & (np.abs(conf - np.float64(np.float32(thr))) <= 1e-5 * conf)
        cm = np.sort(conf[m])[::-1]
        fallback = not (m & (conf.astype(np.float32) > np.float32(thr))).any()
        near_tie = fallback and cm.size >= 2 and cm[0] - cm[1] <= 1e-5 * cm[0]
        # validity in every case
        assert np.all(gd <= masked[sl]) and gd.any() == m.any()
        assert np.array_equal(g["masked_next"][sl], masked[sl] & (1 - gd))
        assert np.array_equal(g["tokens"][sl][gd == 1], g["argmax"][sl][gd == 1]) and np.all(g["tokens"][sl][gd == 0] == -7)
        if near_thr.any() or near_tie:
            continue
        n_exact += 1
        assert np.array_equal(gd, od), (b, gd, od)
        if od.any():
            assert abs(float(g["max_entropy"][b]) - o["max_entropy"][b]) <= 1e-4
            if abs(o["max_entropy"][b] - tau) >= 1e-4:
                assert int(g["decision"][b]) == int(o["decision"][b])
        else:
            assert np.isneginf(g["max_entropy"][b]) and int(g["decision"][b]) == 0
    return n_exact, n_seq


@pytest.mark.parametrize("name,B", [("c1_tiny_fp32", 1), ("c2_llada_l768", 1), ("c3_dream_l768", 2), ("c5_llada_l4096_b8", 8)])
def test_decode_on_benchmark_shapes(name, B):
    w = syn.WORKLOADS[name]
    R = B * w.block
    lg = _logits(R, w.vocab, w.dtype, 60 + w.cfg_id, n_spiked=R // 3)
    rng = np.random.Generator(np.random.PCG64(61))
    masked = (rng.random(R) < 0.7).astype(np.uint8)
    for tau in (1.5, 0.05):
        n_exact, n_seq = _check(lg, w.dtype, w.vocab, masked, 0.9, tau, w.block)
        assert n_exact == n_seq


@pytest.mark.parametrize("dtype", [syn.F32, syn.BF16])
@pytest.mark.parametrize("V,stride,rps,R", [(1000, 1000, 5, 15), (2049, 2056, 64, 128), (40001, 40008, 1, 6), (777, 784, 32, 32)])
def test_decode_ragged_shapes_and_sequence_lengths(dtype, V, stride, rps, R):
    lg = _logits(R, V, dtype, 70 + V % 5, n_spiked=R // 2, stride=stride)
    rng = np.random.Generator(np.random.PCG64(71 + V))
    masked = (rng.random(R) < 0.5).astype(np.uint8)
    _check(lg, dtype, V, masked, 0.9, 1.0, rps)


def test_decode_degenerate_sets():
    V, R, rps = 5000, 64, 32
    lg = _logits(R, V, syn.BF16, 80, n_spiked=0, sigma_hi=1.0)      # flat rows, nobody is confident: one row per sequence
    ones = np.ones(R, np.uint8)
    g = _run(lg, syn.BF16, V, ones, 0.9, 1.5, rps)
    assert g["decoded"][:32].sum() == 1 and g["decoded"][32:].sum() == 1
    _check(lg, syn.BF16, V, ones, 0.9, 1.5, rps)
    g = _run(lg, syn.BF16, V, np.zeros(R, np.uint8), 0.9, 1.5, rps)  # nothing masked: nothing decoded, skip
    assert g["decoded"].sum() == 0 and np.all(np.isneginf(g["max_entropy"])) and g["decision"].tolist() == [0, 0]
    _check(lg, syn.BF16, V, ones, 0.0, 1.5, rps)                     # threshold 0: every masked row is decoded
    g = _run(lg, syn.BF16, V, ones, 0.0, 1.5, rps)
    assert g["decoded"].sum() == R and g["masked_next"].sum() == 0
    half = np.array(([1, 0] * 32), np.uint8)
    _check(_logits(R, V, syn.BF16, 81, n_spiked=R), syn.BF16, V, half, 0.9, 1.5, rps)   # everybody confident, half masked


def test_decode_rejects_long_sequences():
    import paper_2603_18489_b200 as ec

    lg = to_dev(_logits(130, 64, syn.F32, 82, 0))
    with pytest.raises(ec.EcError):
        ec.ec_entropy_gate_decode(lg, 64, 65, torch.ones(130, dtype=torch.uint8, device="cuda"), 0.9, 1.5,
                                  torch.zeros(130, dtype=torch.int32, device="cuda"))
