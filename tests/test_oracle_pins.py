"""Pins for the CPU oracle: it is checked against what the paper's definitions
and plain mathematics fix, never against itself and never against the CUDA path.

Gate (Eq. 1): closed-form entropies, invariances, bounds, fp64 library routines
(scipy, torch), a pure-Python brute force, the skip/recompute flip at tau
(Algorithm 1: E <= tau skips, otherwise recompute).
Attend (Appendix A, partial branch): explicit softmax(QK^T)V matrices, torch's
scaled_dot_product_attention in fp64, degenerate cases with known answers,
permutation invariance, GQA as repeated-head MHA, active rows as a subset of a
full pass.
Refresh (Section 4.2): byte-level checks.
"""
import math
import os

import numpy as np
import pytest

import ec_synth as syn
import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "entropy_closed_forms.txt")


def _gate(x, flags=None, tau=1.5, dtype=syn.F32, rows_per_seq=None, vocab=None, want_probs=False):
    x = np.ascontiguousarray(x, dtype=np.float32)
    if x.ndim == 1:
        x = x[None, :]
    V = x.shape[1] if vocab is None else vocab
    st = syn.encode(x, dtype)
    if flags is None:
        flags = np.ones(x.shape[0], np.uint8)
    return oracle.entropy_gate(st, dtype, V, flags, tau, rows_per_seq, want_probs)


# --------------------------------------------------------------------------- #
# gate: closed forms
# --------------------------------------------------------------------------- #
def _golden_rows():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                kind, V, m, c, H = line.split()
                rows.append((kind, int(V), int(m), float(c), float(H)))
    return rows


@pytest.mark.parametrize("kind,V,m,c,H", _golden_rows())
def test_golden_closed_forms(kind, V, m, c, H):
    """Rows with m entries at value c and the rest at 0 (uniform when c = 0);
    expected entropies stored as text, derived by hand from
    H = ln Z - m c e^c / Z with Z = m e^c + V - m."""
    x = np.zeros(V, np.float32)
    x[:m] = c
    r = _gate(x)
    assert abs(r["entropy"][0] - H) < 1e-9


@pytest.mark.parametrize("V", [2, 7, 1024, 126464, 152064])
def test_uniform_row_is_log_V(V):
    for c in (0.0, -3.25, 17.5):
        r = _gate(np.full(V, c, np.float32))
        # naive fp64 summation over V terms: error bound ~ V * 2^-53 * ln V (2e-10 at V = 152064)
        assert abs(r["entropy"][0] - math.log(V)) < 1e-9
        assert abs(r["conf"][0] - 1.0 / V) < 1e-15
        assert r["argmax"][0] == 0  # all tied: smallest index


def test_one_hot_row_is_zero():
    V = 1024
    x = np.full(V, -np.inf, np.float32)
    x[37] = 2.5
    r = _gate(x)
    assert r["entropy"][0] == 0.0 and r["conf"][0] == 1.0 and r["argmax"][0] == 37
    x = np.zeros(V, np.float32)
    x[1000] = 900.0  # gap >= 800: every other exp underflows to 0 in double
    r = _gate(x)
    assert r["entropy"][0] == 0.0 and r["conf"][0] == 1.0 and r["argmax"][0] == 1000


def test_two_way_tie_is_log2_and_lowest_index_wins():
    V = 513
    x = np.full(V, -np.inf, np.float32)
    x[400] = x[17] = 1.0
    r = _gate(x)
    assert abs(r["entropy"][0] - math.log(2)) < 1e-15
    assert abs(r["conf"][0] - 0.5) < 1e-15
    assert r["argmax"][0] == 17


@pytest.mark.parametrize("V,m,c", [(10, 1, 1.0), (1024, 3, 4.0), (126464, 5, 9.5), (4096, 4095, -2.0)])
def test_spike_rows_closed_form(V, m, c):
    c = float(np.float32(c))
    x = np.zeros(V, np.float32)
    pos = np.random.Generator(np.random.PCG64(V + m)).choice(V, m, replace=False)
    x[pos] = c
    Z = m * math.exp(c) + (V - m)
    H = math.log(Z) - m * c * math.exp(c) / Z
    r = _gate(x)
    assert abs(r["entropy"][0] - H) < 1e-9
    conf = max(math.exp(c), 1.0) / Z
    assert abs(r["conf"][0] - conf) < 1e-11 * conf + 1e-15  # relative: naive summation of Z
    assert r["argmax"][0] == (int(pos.min()) if c > 0 else int(np.setdiff1d(np.arange(V), pos).min()))


def test_pure_python_brute_force_tiny():
    rng = np.random.Generator(np.random.PCG64(5))
    x = (rng.standard_normal((6, 5)) * 3).astype(np.float32)
    r = _gate(x, want_probs=True)
    for i in range(6):
        xs = [float(v) for v in x[i]]
        e = [math.exp(v) for v in xs]  # no max subtraction: a different route
        Z = sum(e)
        p = [v / Z for v in e]
        H = -sum(pi * math.log(pi) for pi in p)
        assert abs(r["entropy"][i] - H) < 1e-13
        assert r["argmax"][i] == max(range(5), key=lambda j: xs[j])
        assert abs(r["conf"][i] - max(p)) < 1e-14
        assert np.allclose(r["probs"][i], p, rtol=0, atol=1e-15)


# --------------------------------------------------------------------------- #
# gate: invariants and library routines
# --------------------------------------------------------------------------- #
def test_shift_invariance_bounds_and_row_sums():
    d = syn.logits_rows(16, 4096, syn.F32, cfg_id=77)
    x = d["logits"]
    r0 = oracle.entropy_gate(x, syn.F32, 4096, np.ones(16, np.uint8), 1.5, want_probs=True)
    # shifting by a power of two keeps fp32 values exactly shifted
    xs = (x.astype(np.float64) + 64.0).astype(np.float32)
    r1 = oracle.entropy_gate(xs, syn.F32, 4096, np.ones(16, np.uint8), 1.5)
    # (x + 64) is not exactly representable for every x; compare with the shifted row's own widening
    exact = np.abs((xs.astype(np.float64) - 64.0) - x.astype(np.float64)).max()
    assert np.abs(r1["entropy"] - r0["entropy"]).max() < 1e-9 + 50 * exact
    H, conf = r0["entropy"], r0["conf"]
    assert (H >= 0).all() and (H <= math.log(4096) + 1e-12).all()
    assert (H >= -np.log(conf) - 1e-12).all()  # H >= min-entropy
    assert (conf >= 1.0 / 4096 - 1e-18).all() and (conf <= 1.0).all()
    assert np.abs(r0["probs"].sum(axis=1) - 1.0).max() < 1e-12
    assert np.array_equal(r0["argmax"], np.argmax(x, axis=1))


def test_exact_shift_invariance():
    rng = np.random.Generator(np.random.PCG64(9))
    x = rng.integers(-40, 40, size=(4, 300)).astype(np.float32) * 0.25  # exact in fp32 after shifting
    r0 = _gate(x)
    r1 = _gate(x + np.float32(1024.0))
    assert np.abs(r0["entropy"] - r1["entropy"]).max() < 1e-12
    assert np.array_equal(r0["argmax"], r1["argmax"])


@pytest.mark.parametrize("dtype", [syn.F32, syn.BF16])
def test_against_scipy_and_torch_fp64(dtype):
    import scipy.special
    import scipy.stats
    import torch

    d = syn.logits_rows(8, 5000, dtype, cfg_id=78, row_stride=5008)
    st = d["logits"]
    flags = np.ones(8, np.uint8)
    r = oracle.entropy_gate(st, dtype, 5000, flags, 1.5, want_probs=True)
    x = syn.decode_f64(st, dtype)[:, :5000]  # padding columns hold a canary and must be ignored
    p = scipy.special.softmax(x, axis=1)
    H = scipy.stats.entropy(p, axis=1)
    assert np.abs(r["entropy"] - H).max() < 1e-11
    assert np.abs(r["probs"] - p).max() < 1e-14
    t = torch.from_numpy(x)
    Ht = torch.distributions.Categorical(logits=t).entropy().numpy()
    assert np.abs(r["entropy"] - Ht).max() < 1e-10
    assert np.array_equal(r["argmax"], np.argmax(x, axis=1))
    assert np.abs(r["conf"] - p.max(axis=1)).max() < 1e-14
    assert abs(r["max_entropy"][0] - H.max()) < 1e-11


def test_small_sigma_gaussian_rows_statistics():
    """iid N(0, s^2) logits with s^2 << 2 ln V: H = ln V - s^2/2 up to sampling noise."""
    V, s = 126464, 0.5
    d = syn.logits_rows(4, V, syn.F32, cfg_id=79, sigma_lo=s, sigma_hi=s)
    r = oracle.entropy_gate(d["logits"], syn.F32, V, np.ones(4, np.uint8), 1.5)
    assert np.abs(r["entropy"] - (math.log(V) - s * s / 2)).max() < 5e-3


def test_bf16_widening_is_exact():
    rng = np.random.Generator(np.random.PCG64(3))
    x = (rng.standard_normal((3, 257)) * 5).astype(np.float32)
    xb = syn.bf16_bits_to_f32(syn.f32_to_bf16_bits(x))  # bf16-representable values as fp32
    a = oracle.entropy_gate(syn.f32_to_bf16_bits(x), syn.BF16, 257, np.ones(3, np.uint8), 1.0)
    b = oracle.entropy_gate(xb, syn.F32, 257, np.ones(3, np.uint8), 1.0)
    for key in ("entropy", "conf", "argmax", "max_entropy", "decision"):
        assert np.array_equal(a[key], b[key])
    # the bf16 encoder itself: round-to-nearest-even on known patterns
    probe = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.3895313892515355e38], np.float32)
    bits = syn.f32_to_bf16_bits(probe)
    assert list(bits) == [0x3F80, 0x3F80, 0x3F82, 0xC020, 0x7F7F]
    # 1 + 2^-8 lies halfway between 0x3F80 and 0x3F81 -> even (0x3F80);
    # 1 + 3*2^-8 lies halfway between 0x3F81 and 0x3F82 -> even (0x3F82).


# --------------------------------------------------------------------------- #
# gate: masked max and the decision rule
# --------------------------------------------------------------------------- #
def test_gate_flips_exactly_at_tau():
    V = 64
    x = np.full((2, V), -np.inf, np.float32)
    x[0, [3, 9]] = 0.0        # H = ln 2
    x[1, 5] = 0.0             # H = 0
    E = math.log(2.0)
    tau_hi = np.float32(E)                       # fp32(ln 2) = 0.69314718246... > ln 2
    assert float(tau_hi) > E
    tau_lo = np.nextafter(tau_hi, np.float32(-np.inf))
    assert float(tau_lo) < E
    r = _gate(x, tau=float(tau_hi))
    assert r["decision"][0] == oracle.SKIP and abs(r["max_entropy"][0] - E) < 1e-15
    r = _gate(x, tau=float(tau_lo))
    assert r["decision"][0] == oracle.RECOMPUTE
    # exact equality E == tau skips: four-way tie has H = ln 4; use a row whose H is 0 and tau = 0
    r = _gate(x[1:], tau=0.0)
    assert r["max_entropy"][0] == 0.0 and r["decision"][0] == oracle.SKIP
    r = _gate(x[1:], tau=float(np.nextafter(np.float32(0), np.float32(-1))))
    assert r["decision"][0] == oracle.RECOMPUTE


def test_unflagged_rows_do_not_count_and_empty_set_skips():
    V = 128
    x = np.zeros((4, V), np.float32)          # rows 0..3 uniform: H = ln 128 = 4.85
    x[1, 0] = 50.0                             # row 1 peaked: H ~ 0
    flags = np.array([0, 1, 0, 0], np.uint8)
    r = _gate(x, flags=flags, tau=1.5)
    assert r["decision"][0] == oracle.SKIP and r["max_entropy"][0] < 1e-15
    flags[:] = 0
    r = _gate(x, flags=flags, tau=-5.0)
    assert r["max_entropy"][0] == -np.inf and r["decision"][0] == oracle.SKIP
    flags[:] = [0, 1, 1, 0]
    r = _gate(x, flags=flags, tau=1.5)
    assert r["decision"][0] == oracle.RECOMPUTE and abs(r["max_entropy"][0] - math.log(V)) < 1e-12


def test_per_sequence_decisions():
    V = 32
    x = np.zeros((6, V), np.float32)
    x[0:3, 0] = 60.0                           # sequence 0: all peaked
    flags = np.ones(6, np.uint8)
    r = _gate(x, flags=flags, tau=1.5, rows_per_seq=3)
    assert list(r["decision"]) == [oracle.SKIP, oracle.RECOMPUTE]
    assert r["max_entropy"].shape == (2,)
    with pytest.raises(ValueError):
        _gate(x, flags=flags, rows_per_seq=4)


# --------------------------------------------------------------------------- #
# attend
# --------------------------------------------------------------------------- #
def _np_attention(q, k, v, scale):
    """softmax(Q K^T * scale) V with explicit matrices, fp64.  q [B,n,Hq,D]; k,v [B,Hkv,L,D]."""
    B, n, Hq, D = q.shape
    Hkv = k.shape[1]
    g = Hq // Hkv
    out = np.empty((B, n, Hq, D))
    for b in range(B):
        for h in range(Hq):
            S = (q[b, :, h, :] @ k[b, h // g].T) * scale
            S = S - S.max(axis=1, keepdims=True)
            P = np.exp(S)
            P /= P.sum(axis=1, keepdims=True)
            out[b, :, h, :] = P @ v[b, h // g]
    return out


@pytest.mark.parametrize("dtype", [syn.F32, syn.BF16])
@pytest.mark.parametrize("Hq,Hkv", [(4, 4), (6, 2)])
def test_full_pass_equals_matrix_attention_and_sdpa(dtype, Hq, Hkv):
    import torch

    w = syn.small_attn_workload(dtype, 2, Hq, Hkv, 16, 24)
    t = syn.attn_inputs(w, 24, std_qk=1.0, std_v=1.0)
    O = oracle.attend(t["q"], t["k_cache"], t["v_cache"], dtype)
    q, k, v = (syn.decode_f64(t[n], dtype) for n in ("q", "k_cache", "v_cache"))
    ref = _np_attention(q, k, v, 1.0 / math.sqrt(16))
    assert np.abs(O - ref).max() < 1e-13
    g = Hq // Hkv
    tq = torch.from_numpy(q).permute(0, 2, 1, 3)
    tk = torch.from_numpy(k).repeat_interleave(g, dim=1)
    tv = torch.from_numpy(v).repeat_interleave(g, dim=1)
    sd = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=False)
    assert np.abs(O - sd.permute(0, 2, 1, 3).numpy()).max() < 1e-12
    # explicit scale
    O2 = oracle.attend(t["q"], t["k_cache"], t["v_cache"], dtype, scale=0.3)
    assert np.abs(O2 - _np_attention(q, k, v, 0.3)).max() < 1e-13


def test_degenerate_cases_with_known_answers():
    w = syn.small_attn_workload(syn.F32, 1, 2, 2, 8, 20)
    t = syn.attn_inputs(w, 20, std_qk=1.0, std_v=1.0)
    q, k, v = t["q"], t["k_cache"].copy(), t["v_cache"].copy()
    # V constant over keys -> O is that constant vector
    vc = v.copy()
    vc[:] = vc[:, :, :1, :]
    O = oracle.attend(q, k, vc, syn.F32)
    for h in range(2):
        assert np.abs(O[0, :, h, :] - vc[0, h, 0, :].astype(np.float64)).max() < 1e-14
    # K constant over keys -> uniform weights -> O = mean of V
    kc = k.copy()
    kc[:] = kc[:, :, :1, :]
    O = oracle.attend(q, kc, v, syn.F32)
    for h in range(2):
        assert np.abs(O[0, :, h, :] - v[0, h].astype(np.float64).mean(axis=0)).max() < 1e-14
    # one dominant key (score + 800 above the rest) -> O = that key's V row
    qd = np.zeros_like(q)
    qd[..., 0] = 1.0
    kd = np.zeros_like(k)
    kd[0, :, 13, 0] = 800.0
    O = oracle.attend(qd, kd, v, syn.F32, scale=1.0)
    for h in range(2):
        assert np.array_equal(O[0, 5, h, :], v[0, h, 13, :].astype(np.float64))
    # convexity: each output lies within the range of V over keys
    O = oracle.attend(q, k, v, syn.F32)
    for h in range(2):
        lo, hi = v[0, h].min(axis=0), v[0, h].max(axis=0)
        assert (O[0, :, h, :] >= lo - 1e-12).all() and (O[0, :, h, :] <= hi + 1e-12).all()


def test_key_permutation_invariance_and_q_k_not_swapped():
    w = syn.small_attn_workload(syn.F32, 1, 3, 3, 8, 17)
    t = syn.attn_inputs(w, 17, std_qk=1.5, std_v=1.0)
    perm = np.random.Generator(np.random.PCG64(1)).permutation(17)
    O0 = oracle.attend(t["q"], t["k_cache"], t["v_cache"], syn.F32)
    O1 = oracle.attend(t["q"], np.ascontiguousarray(t["k_cache"][:, :, perm]),
                       np.ascontiguousarray(t["v_cache"][:, :, perm]), syn.F32)
    assert np.abs(O0 - O1).max() < 1e-13
    # permuting only K (not V) must change the result: keys and values are paired by position
    O2 = oracle.attend(t["q"], np.ascontiguousarray(t["k_cache"][:, :, perm]), t["v_cache"], syn.F32)
    assert np.abs(O0 - O2).max() > 1e-3


def test_gqa_equals_mha_on_repeated_heads():
    w = syn.small_attn_workload(syn.BF16, 2, 8, 2, 16, 12)
    t = syn.attn_inputs(w, 12, std_qk=1.0, std_v=1.0)
    O = oracle.attend(t["q"], t["k_cache"], t["v_cache"], syn.BF16)
    kr = np.ascontiguousarray(np.repeat(t["k_cache"], 4, axis=1))
    vr = np.ascontiguousarray(np.repeat(t["v_cache"], 4, axis=1))
    Om = oracle.attend(t["q"], kr, vr, syn.BF16)
    assert np.array_equal(O, Om)


def test_active_rows_are_a_subset_of_the_full_pass():
    w = syn.small_attn_workload(syn.F32, 2, 4, 2, 8, 32, block=4)
    t = syn.attn_inputs(w, 32, std_qk=1.0, std_v=1.0)
    full = oracle.attend(t["q"], t["k_cache"], t["v_cache"], syn.F32)
    rows = [30, 2, 17]
    sub = oracle.attend(t["q"], t["k_cache"], t["v_cache"], syn.F32, row_sel=rows)
    assert np.array_equal(sub, full[:, rows])
    qs = np.ascontiguousarray(t["q"][:, rows])
    sub2 = oracle.attend(qs, t["k_cache"], t["v_cache"], syn.F32)
    assert np.array_equal(sub2, full[:, rows])


def test_layer_step_refreshes_before_attending():
    w = syn.small_attn_workload(syn.F32, 2, 2, 2, 8, 16, block=4)
    t = syn.attn_inputs(w, 6, std_qk=1.0, std_v=1.0, k_recent=2)
    idx = t["active_idx"]
    kc, vc = t["k_cache"].copy(), t["v_cache"].copy()
    O = oracle.refresh_and_attend(t["q"], t["k_new"], t["v_new"], kc, vc, idx, syn.F32)
    # manual patch with numpy indexing, then matrix attention
    km, vm = t["k_cache"].copy(), t["v_cache"].copy()
    for b in range(2):
        for i in range(6):
            km[b, :, idx[b, i], :] = t["k_new"][b, i]
            vm[b, :, idx[b, i], :] = t["v_new"][b, i]
    assert np.array_equal(kc, km) and np.array_equal(vc, vm)
    ref = _np_attention(t["q"].astype(np.float64), km.astype(np.float64), vm.astype(np.float64),
                        1 / math.sqrt(8))
    assert np.abs(O - ref).max() < 1e-13
    stale = oracle.attend(t["q"], t["k_cache"], t["v_cache"], syn.F32)
    assert np.abs(O - stale).max() > 1e-3  # attending over the stale cache is a different result


# --------------------------------------------------------------------------- #
# refresh
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("dtype", [syn.F32, syn.BF16])
def test_refresh_bytes(dtype):
    B, Hkv, L, D, n = 2, 3, 19, 8, 5
    w = syn.Workload(91, "r", dtype, B, 3, Hkv, D, 9, 10, 3, 2, 16)
    t = syn.attn_inputs(w, n)
    idx = syn.arbitrary_active_idx(B, L, n, seed=4)
    k0, v0 = t["k_cache"].copy(), t["v_cache"].copy()
    k, v = k0.copy(), v0.copy()
    oracle.kv_refresh(k, v, t["k_new"], t["v_new"], idx, dtype)
    touched = np.zeros((B, L), bool)
    for b in range(B):
        for i in range(n):
            assert np.array_equal(k[b, :, idx[b, i], :], t["k_new"][b, i])
            assert np.array_equal(v[b, :, idx[b, i], :], t["v_new"][b, i])
            touched[b, idx[b, i]] = True
    for b in range(B):
        assert np.array_equal(k[b][:, ~touched[b]], k0[b][:, ~touched[b]])
        assert np.array_equal(v[b][:, ~touched[b]], v0[b][:, ~touched[b]])
    k2, v2 = k.copy(), v.copy()
    oracle.kv_refresh(k2, v2, t["k_new"], t["v_new"], idx, dtype)  # idempotent
    assert np.array_equal(k2, k) and np.array_equal(v2, v)
    bad = idx.copy()
    bad[1, 2] = L
    with pytest.raises(ValueError):
        oracle.kv_refresh(k2, v2, t["k_new"], t["v_new"], bad, dtype)
    assert np.array_equal(k2, k)  # nothing written on error


def test_identity_refresh_is_a_transposed_copy():
    w = syn.small_attn_workload(syn.BF16, 2, 4, 2, 8, 12)
    t = syn.attn_inputs(w, 12)
    assert t["active_idx"] is None
    k, v = t["k_cache"].copy(), t["v_cache"].copy()
    oracle.kv_refresh(k, v, t["k_new"], t["v_new"], None, syn.BF16)
    assert np.array_equal(k, np.transpose(t["k_new"], (0, 2, 1, 3)))
    assert np.array_equal(v, np.transpose(t["v_new"], (0, 2, 1, 3)))


# --------------------------------------------------------------------------- #
# Recent-token selection (Eq. 2-3) and the step bookkeeping of Appendix A
# --------------------------------------------------------------------------- #
def _parse_h(s):
    return np.array([-np.inf if x.strip() == "n" else float(x) for x in s.split(",")])


def test_recent_selection_matches_the_hand_worked_cases():
    path = os.path.join(os.path.dirname(__file__), "golden", "recent_selection_worked.txt")
    n = 0
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        h, k, t, dt, exp = [x.strip() for x in line.split("|")]
        want = [int(x) for x in exp.split(",")] if exp else []
        got = oracle.select_recent(_parse_h(h), int(k), int(t), int(dt)).tolist()
        assert got == want, line
        n += 1
    assert n >= 9


def test_recent_selection_threshold_equals_brute_force_over_all_k_subsets():
    """Eq. 3 literally: K maximises the sum of H over all subsets of size k (never-decoded entries count as a very
    negative number so that they are taken last); the minimum over K is unique even when K is not."""
    import itertools

    rng = np.random.Generator(np.random.PCG64(31))
    for trial in range(60):
        n = int(rng.integers(3, 9))
        H = rng.integers(0, 5, size=n).astype(np.float64)
        H[rng.random(n) < 0.35] = -np.inf
        k = int(rng.integers(1, n + 1))
        t, dt = 5, int(rng.integers(0, 6))
        big = np.where(np.isfinite(H), H, -1e9)
        best = max(itertools.combinations(range(n), k), key=lambda s: sum(big[list(s)]))
        min_k = min(H[list(best)])
        tau_r = max(min_k, t - dt)
        want = [i for i in range(n) if H[i] >= tau_r]
        assert oracle.select_recent(H, k, t, dt).tolist() == want


def test_recent_selection_properties():
    rng = np.random.Generator(np.random.PCG64(32))
    H = rng.integers(1, 40, size=300).astype(np.float64)
    H[rng.random(300) < 0.5] = -np.inf
    t = 40
    assert oracle.select_recent(H, 0, t, 10).size == 0                       # no budget, nothing selected
    prev = -1
    for k in (1, 2, 8, 64, 150, 300):                                         # a larger budget never selects less
        R = oracle.select_recent(H, k, t, 40)
        assert R.size >= min(k, int(np.isfinite(H).sum())) and R.size >= prev
        assert np.all(np.diff(R) > 0) and np.all(np.isfinite(H[R]))
        prev = R.size
    for dt in range(0, 12):                                                   # never older than the last full pass
        R = oracle.select_recent(H, 64, t, dt)
        assert np.all(H[R] >= t - dt)
    R0 = oracle.select_recent(H, 64, t, 0)
    assert set(R0.tolist()) == set(np.flatnonzero(H == t).tolist())          # dt = 0: only this step's tokens


def test_step_bookkeeping_follows_appendix_a_order():
    H = np.full(12, -np.inf)
    # step t = 1 (a full pass happened, dt = 0): positions 4, 5 decoded, gate says skip
    R, skip, dt, t = oracle.step_bookkeeping(H, 1, 0, [4, 5], oracle.SKIP, k=2)
    assert H[4] == 1 and H[5] == 1 and R.tolist() == [4, 5] and skip and dt == 1 and t == 2
    # step 2 (partial), position 6 decoded, gate says skip: K = {6, one of 4/5}, min 1, tau_R = max(1, 2 - 1) = 1
    R, skip, dt, t = oracle.step_bookkeeping(H, t, dt, [6], oracle.SKIP, k=2)
    assert R.tolist() == [4, 5, 6] and dt == 2 and t == 3
    # step 3, position 7 decoded, gate says recompute: the selection still uses dt = 2 (tau_R = max(2, 1) = 2)
    R, skip, dt, t = oracle.step_bookkeeping(H, t, dt, [7], oracle.RECOMPUTE, k=2)
    assert R.tolist() == [6, 7] and not skip and dt == 0 and t == 4
    rows = oracle.partial_step_rows(4, 4, np.array([1, 5, 9, 6]))
    assert rows.tolist() == [4, 5, 6, 7, 1, 9]


# --------------------------------------------------------------------------- #
# Confidence-based parallel decoding behind the gate (Section 2.1; threshold 0.9 in Section 5.1)
# --------------------------------------------------------------------------- #
def test_confident_rows_are_decoded_and_otherwise_the_single_best_masked_row():
    f = lambda c, m, thr=0.9: oracle.decode_confident(np.array(c), np.array(m), thr).tolist()
    assert f([0.95, 0.5, 0.91, 0.99], [1, 1, 0, 1]) == [1, 0, 0, 1]          # row 2 is confident but not masked
    assert f([0.3, 0.8, 0.85, 0.85], [1, 0, 1, 1]) == [0, 0, 1, 0]           # nobody above 0.9: best masked row, first of the tie
    assert f([0.3, 0.95, 0.2, 0.1], [1, 0, 1, 1]) == [1, 0, 0, 0]            # the confident row is unmasked: fallback among the masked
    assert f([0.5, 0.6], [0, 0]) == [0, 0]                                   # nothing left to decode
    assert f([np.float32(0.9), 0.2], [1, 1]) == [1, 0]                       # exactly the threshold is not above it: chosen only as the best
    assert f([np.float32(0.9), np.nextafter(np.float32(0.9), np.float32(1))], [1, 1]) == [0, 1]
    assert f([0.2, 0.4, 0.3], [1, 1, 1], thr=0.25) == [0, 1, 1]


def test_gate_with_its_own_decoded_set_on_spike_and_flat_rows():
    """Rows with one logit c above V - 1 zeros: conf = e^c / Z, H = ln Z - c e^c / Z, Z = e^c + V - 1 (closed form)."""
    V = 16
    cs = [10.0, 0.0, 6.0, 10.0, 2.0, 0.0]
    lg = np.zeros((6, V), np.float32)
    for r, c in enumerate(cs):
        lg[r, (3 * r) % V] = c
    Z = [math.exp(c) + V - 1 for c in cs]
    conf = [math.exp(c) / z for c, z in zip(cs, Z)]
    H = [math.log(z) - c * math.exp(c) / z for c, z in zip(cs, Z)]
    assert conf[0] > 0.9 and conf[2] > 0.9 and conf[4] < 0.9
    masked = np.array([1, 1, 1, 0, 1, 1], np.uint8)                           # row 3 was decoded earlier
    o = oracle.entropy_gate_decode(lg, oracle.F32, V, masked, 0.9, tau=0.02, rows_per_seq=6)
    assert o["decoded"].tolist() == [1, 0, 1, 0, 0, 0]
    assert o["masked_next"].tolist() == [0, 1, 0, 0, 1, 1]
    assert o["tokens"].tolist() == [0, -1, 6, -1, -1, -1]
    assert abs(o["max_entropy"][0] - max(H[0], H[2])) < 1e-12 and o["max_entropy"][0] == pytest.approx(H[2])
    assert o["decision"].tolist() == [1 if H[2] > 0.02 else 0]
    # two sequences of three rows: the second has no confident masked row -> its best masked row (row 4) alone
    o = oracle.entropy_gate_decode(lg, oracle.F32, V, np.array([1, 1, 1, 0, 1, 1], np.uint8), 0.9, tau=3.0, rows_per_seq=3)
    assert o["decoded"].tolist() == [1, 0, 1, 0, 1, 0]
    assert o["max_entropy"][1] == pytest.approx(H[4]) and o["decision"].tolist() == [0, 0]


def test_decode_invariants_on_random_rows():
    rng = np.random.Generator(np.random.PCG64(77))
    for trial in range(50):
        n = int(rng.integers(1, 40))
        conf = rng.random(n) ** 0.3
        masked = (rng.random(n) < 0.6).astype(np.uint8)
        d = oracle.decode_confident(conf, masked, 0.9)
        assert np.all(d <= masked)                                            # only masked rows are decoded
        assert d.any() == masked.any()                                        # a step decodes something while anything is masked
        above = (masked == 1) & (conf.astype(np.float32) > np.float32(0.9))
        if above.any():
            assert np.array_equal(d.astype(bool), above)
        else:
            assert d.sum() == int(masked.any())


# --------------------------------------------------------------------------- #
# The three candidate gate metrics (Section 5.3)
# --------------------------------------------------------------------------- #
def test_gate_metrics_on_hand_worked_rows():
    ent = np.array([0.5, 2.0, 0.25, 1.0, 3.0, 0.125])
    conf = np.array([0.9, 0.3, 0.95, 0.6, 0.1, 0.99])
    flags = np.array([1, 0, 1, 1, 0, 0], np.uint8)
    m = oracle.gate_metrics(ent, conf, flags, 6)
    assert m["max_entropy"].tolist() == [1.0] and m["entropy_sum"].tolist() == [1.75] and m["max_conf"].tolist() == [0.95]
    m = oracle.gate_metrics(ent, conf, flags, 3)                      # two sequences of three rows
    assert m["max_entropy"].tolist() == [0.5, 1.0] and m["entropy_sum"].tolist() == [0.75, 1.0]
    assert m["max_conf"].tolist() == [0.95, 0.6]
    m = oracle.gate_metrics(ent, conf, np.zeros(6, np.uint8), 6)      # nothing decoded
    assert np.isneginf(m["max_entropy"][0]) and m["entropy_sum"][0] == 0.0 and np.isneginf(m["max_conf"][0])


def test_gate_metrics_agree_with_the_gate_and_with_each_other():
    V, R = 300, 24
    d = syn.logits_rows(R, V, syn.F32, cfg_id=88)
    flags = syn.decoded_flags(R, 3, 8, cfg_id=88)
    g = oracle.entropy_gate(d["logits"], syn.F32, V, flags, 1.0, 8)
    m = oracle.gate_metrics(g["entropy"], g["conf"], flags, 8)
    assert np.array_equal(m["max_entropy"], g["max_entropy"])        # metric (1) is Eq. 1's E
    for b in range(3):
        n = int(flags[8 * b:8 * b + 8].sum())
        assert m["max_entropy"][b] <= m["entropy_sum"][b] + 1e-15 <= n * m["max_entropy"][b] + 1e-12
        assert 1.0 / V <= m["max_conf"][b] <= 1.0
        # the most confident decoded row has at most -ln(conf) ... entropy bound from below: H >= -ln(max p)
        assert m["max_entropy"][b] >= -math.log(m["max_conf"][b]) - 1e-12 or n > 1


# --------------------------------------------------------------------------- #
# Sliding-window decoding (Section 2.1)
# --------------------------------------------------------------------------- #
def test_sliding_window_advances_and_keeps_its_size():
    masked = np.array([0, 0, 1, 1, 1, 1, 1, 1, 1, 1], np.uint8)           # two prompt positions, eight to generate
    H = np.full(10, -np.inf)
    win = oracle.sliding_window_rows(masked, 4)
    assert win.tolist() == [2, 3, 4, 5]
    # step 1: rows 1 and 3 of the window (positions 3 and 5) are decoded; gate says skip
    rows, skip, dt, t = oracle.sliding_step_bookkeeping(H, masked, 1, 0, win, np.array([0, 1, 0, 1], np.uint8), oracle.SKIP, 2, 4)
    assert masked.tolist() == [0, 0, 1, 0, 1, 0, 1, 1, 1, 1] and H[3] == 1 and H[5] == 1
    assert rows.tolist() == [2, 4, 6, 7, 3, 5] and skip and dt == 1 and t == 2      # window no longer contiguous, then R
    # step 2: row 0 (position 2) decoded; K = {2 (H = 2), one of H = 1}, min 1, tau_R = max(1, 2 - 1) = 1
    rows, skip, dt, t = oracle.sliding_step_bookkeeping(H, masked, t, dt, rows[:4], np.array([1, 0, 0, 0], np.uint8), oracle.SKIP, 2, 4)
    assert rows.tolist() == [4, 6, 7, 8, 2, 3, 5] and dt == 2
    # near the end fewer masked positions remain than the window holds
    masked[:] = 0
    masked[9] = 1
    assert oracle.sliding_window_rows(masked, 4).tolist() == [9]


def test_sliding_window_and_recent_set_never_overlap():
    rng = np.random.Generator(np.random.PCG64(91))
    L, window, k = 200, 16, 5
    masked = np.ones(L, np.uint8); masked[:40] = 0
    H = np.full(L, -np.inf)
    t, dt = 1, 0
    rows = oracle.sliding_window_rows(masked, window)
    for step in range(12):
        flags = (rng.random(window) < 0.25).astype(np.uint8)
        win = rows[:window]
        rows, skip, dt, t = oracle.sliding_step_bookkeeping(H, masked, t, dt, win, flags, int(rng.integers(0, 2)), k, window)
        nxt, R = rows[:window], rows[window:]
        assert nxt.size == window and np.all(np.diff(nxt) > 0) and np.all(masked[nxt] == 1)
        assert np.all(np.isfinite(H[R])) and not set(nxt.tolist()) & set(R.tolist())
        assert int(masked.sum()) == 160 - int(np.isfinite(H).sum())
