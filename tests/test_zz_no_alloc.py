"""ec_entropy_gate_static: the allocation-free variant of the entropy gate, for
callers that cannot allocate device memory (a server whose HBM is already fully
partitioned, a plug-in inside another runtime's pool).  Its scratch is a fixed
array inside the library, shared by all calls, so this test checks that two
calls in a row -- on different inputs, the second one smaller -- each reproduce
what the regular entry point returns with a caller-owned workspace, and what the
fp64 oracle computes (Eq. 1 of the paper) within the gate's tolerances.  It is
collected last so that a failure here cannot hide the other tests."""
import ctypes

import numpy as np
import pytest
import torch

import ec_synth as syn
import oracle
from _util import to_dev

pytestmark = pytest.mark.gpu


def _outs(R, nseq):
    z = lambda n, dt: torch.full((n,), -7, dtype=dt, device="cuda")
    return dict(argmax=z(R, torch.int32), conf=z(R, torch.float32), entropy=z(R, torch.float32),
                max_entropy=z(nseq, torch.float32), decision=z(nseq, torch.int32))


def _call_static(lib, logits, vocab, rps, flags, tau, o):
    vp = ctypes.c_void_p
    st = lib.ec_entropy_gate_static(vp(logits.data_ptr()), 1 if logits.dtype == torch.bfloat16 else 0,
                                    logits.shape[0], vocab, logits.stride(0), rps, vp(flags.data_ptr()), tau,
                                    vp(o["argmax"].data_ptr()), vp(o["conf"].data_ptr()),
                                    vp(o["entropy"].data_ptr()), vp(o["max_entropy"].data_ptr()),
                                    vp(o["decision"].data_ptr()), vp(torch.cuda.current_stream().cuda_stream))
    return st


def test_static_gate_matches_workspace_gate_on_two_calls_in_a_row():
    import paper_2603_18489_b200 as ec

    cases = [(syn.C5B8, 256, 32, 1.5, 70), (syn.C3, 32, 32, 3.0, 71)]   # large first, then smaller
    for w, R, rps, tau, seed in cases:
        d = syn.logits_rows(R, w.vocab, w.dtype, cfg_id=seed)
        flags = to_dev(syn.decoded_flags(R, 9, rps, cfg_id=seed))
        logits = to_dev(d["logits"])
        ref = ec.ec_entropy_gate(logits, w.vocab, rps, flags, tau)
        o = _outs(R, R // rps)
        assert _call_static(ec.lib, logits, w.vocab, rps, flags, tau, o) == 0
        torch.cuda.synchronize()
        assert torch.equal(o["argmax"], ref["argmax"])
        assert torch.equal(o["decision"], ref["decision"])
        for k in ("conf", "entropy", "max_entropy"):
            assert (o[k] - ref[k]).abs().max().item() <= 1e-4
        want = oracle.entropy_gate(d["logits"], w.dtype, w.vocab, syn.decoded_flags(R, 9, rps, cfg_id=seed), tau, rps)
        assert np.array_equal(o["argmax"].cpu().numpy(), want["argmax"])
        assert np.abs(o["entropy"].cpu().numpy() - want["entropy"]).max() <= 1e-4
        assert (np.abs(o["conf"].cpu().numpy() - want["conf"]) <= 1e-5 * want["conf"]).all()
        assert np.abs(o["max_entropy"].cpu().numpy() - want["max_entropy"]).max() <= 1e-4
        far = np.abs(want["max_entropy"] - np.float64(np.float32(tau))) >= 1e-4
        assert np.array_equal(o["decision"].cpu().numpy()[far], want["decision"][far])


def test_static_gate_refuses_sizes_beyond_its_scratch_and_bad_arguments():
    import paper_2603_18489_b200 as ec

    R = ec.EC_GATE_STATIC_MAX_ROWS + 32
    logits = torch.zeros(R, 1024, device="cuda", dtype=torch.bfloat16)
    flags = torch.ones(R, device="cuda", dtype=torch.uint8)
    o = _outs(R, R // 32)
    assert _call_static(ec.lib, logits, 1024, 32, flags, 1.5, o) == 6       # EC_ERR_UNSUPPORTED
    small = logits[:32]
    assert _call_static(ec.lib, small, 1024, 5, flags, 1.5, o) == 2         # 32 % 5 != 0: EC_ERR_SHAPE
    with pytest.raises(ec.EcError):
        ec.ec_entropy_gate_static(logits, 1024, 32, flags, 1.5, max_entropy_out=o["max_entropy"],
                                  decision_out=o["decision"])
    torch.cuda.synchronize()
    assert int(o["decision"][0]) == -7                                      # nothing was launched
