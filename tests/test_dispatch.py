"""Which kernel ec_attend picks for each benchmark shape (host-only query, no launch).  The parity tests in
test_gpu_attend.py / test_gpu_config5.py run these very shapes against the oracle; this table pins the kernel
behind each of them, so a change of the dispatch cannot leave a kernel without a parity test unnoticed.
The plans assume 148 SMs (the B200's count, also the library's default when no device can be queried); cluster sizes
are not pinned here, because with a device present the library asks the runtime how many clusters stay resident."""
import pytest

import ec_synth as syn

# (workload, batch override, active rows) -> kernel family with its instantiation, on the skip step
SKIP_STEP = [
    ("c2_llada_l768", None, 34, "attend_skip_keys_kernel<48>"),
    ("c3_dream_l768", None, 34, "attend_skip_keys_kernel<48>"),
    ("c4_llada_l2048", None, 33, "attend_skip_keys_kernel<48>"),
    ("c4_llada_l2048", None, 40, "attend_skip_keys_kernel<48>"),
    ("c5_llada_l4096", None, 34, "attend_skip_keys_kernel<48>"),
    ("c5_llada_l4096", 2, 34, "attend_skip_keys_kernel<48>"),
    ("c5_llada_l4096_b8", None, 34, "attend_skip_kernel<1>"),       # beyond one wave of one-CTA-per-SM clusters
    ("c5_llada_l4096", 5, 34, "attend_skip_kernel<1>"),
    ("c4_dream_l2048", None, 34, "attend_skip_keys_kernel<48>"),
    ("c5_dream_l4096", None, 34, "attend_skip_keys_kernel<48>"),
    ("c5_llada_l4096", None, 96, "attend_skip_keys_kernel<96>"),    # the paper's default budget k = 64
    ("c5_llada_l4096_b8", None, 96, "attend_skip_kernel<1>"),
    ("c5_dream_l4096", None, 96, "attend_skip_keys_kernel<96>"),
    ("c1_tiny_fp32", None, 34, "refresh_kernel + attend_f32_kernel"),
]

RECOMPUTE_STEP = [
    ("c1_tiny_fp32", None, "refresh_kernel + attend_f32_kernel"),
    ("c2_llada_l768", None, "attend_dense_kernel"),
    ("c3_dream_l768", None, "attend_dense_kernel"),
    ("c4_llada_l2048", None, "attend_dense_kernel"),
    ("c5_llada_l4096", None, "attend_dense_kernel"),
    ("c5_llada_l4096_b8", None, "attend_dense_kernel"),
    ("c4_dream_l2048", None, "attend_dense_kernel"),
    ("c5_dream_l4096", None, "attend_dense_kernel"),
]


def _desc(name, batch):
    import paper_2603_18489_b200 as ec

    w = syn.WORKLOADS[name]
    return ec, ec.make_desc(batch or w.batch, w.ctx_len, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype), w


@pytest.mark.parametrize("name,batch,n,kernel", SKIP_STEP)
def test_kernel_of_each_benchmark_skip_step(name, batch, n, kernel):
    ec, d, w = _desc(name, batch)
    got = ec.ec_attend_kernel_name(d, n, True, True)
    assert got.startswith(kernel), got
    if "grid=" in got:      # the cluster splits the key tiles; the grid's second dimension covers every (sequence, head)
        gx, gy = (int(v) for v in got.split("grid=(")[1].split(")")[0].split(","))
        assert gy % ((batch or w.batch) * w.n_kv_heads) == 0 and f"cluster={gx}" in got


@pytest.mark.parametrize("name,batch,kernel", RECOMPUTE_STEP)
def test_kernel_of_each_benchmark_recompute_step(name, batch, kernel):
    ec, d, w = _desc(name, batch)
    got = ec.ec_attend_kernel_name(d, w.ctx_len, True, False)
    assert got.startswith(kernel), got


def test_other_instantiations_and_fallbacks_are_reachable():
    """Every kernel (and template instantiation) of the attention path, with a shape that reaches it; each of
    these shapes has a parity case in test_gpu_attend.py."""
    import paper_2603_18489_b200 as ec

    def name(B, L, Hq, Hkv, D, dtype, n, idx=True):
        return ec.ec_attend_kernel_name(ec.make_desc(B, L, Hq, Hkv, D, dtype), n, True, idx)

    assert name(2, 1000, 8, 8, 128, syn.BF16, 56).startswith("attend_skip_keys_kernel<64>")
    assert name(2, 333, 6, 3, 128, syn.BF16, 100).startswith("attend_skip_keys_kernel<64>")  # 200 packed rows
    assert name(1, 640, 4, 4, 128, syn.BF16, 256).startswith("attend_skip_keys_kernel<96>")  # three row chunks
    assert "fresh_tiles=1" in name(1, 768, 32, 32, 128, syn.BF16, 34)      # the refreshed rows are attended as one extra tile
    assert "fresh_tiles=2" in name(1, 4096, 32, 32, 128, syn.BF16, 160)
    assert "fresh_tiles=0" in ec.ec_attend_kernel_name(ec.make_desc(1, 768, 32, 32, 128, syn.BF16), 34, False, True)
    assert name(2, 768, 32, 32, 128, syn.BF16, 128).startswith("attend_skip_kernel<1> grid=(4,64) cluster=4")
    assert name(3, 768, 32, 32, 128, syn.BF16, 128).startswith("attend_skip_kernel<1> grid=(3,96) cluster=3")
    assert name(2, 768, 32, 32, 128, syn.BF16, 160).startswith("attend_skip_kernel<2> grid=(2,64) cluster=2")
    assert name(8, 4096, 32, 32, 128, syn.BF16, 200).startswith("attend_skip_kernel<2> grid=(1,256) cluster=1")
    assert name(2, 65, 6, 3, 128, syn.BF16, 65, idx=False).startswith("attend_skip_keys_kernel<96>")
    assert name(2, 259, 4, 2, 128, syn.BF16, 259, idx=False) == "refresh_kernel + attend_tc_kernel"
    assert name(2, 130, 6, 3, 64, syn.BF16, 17) == "refresh_kernel + attend_mma_kernel"
    assert name(2, 130, 6, 3, 64, syn.F32, 17) == "refresh_kernel + attend_f32_kernel"
    # the dense kernel cuts the units of its last, partial wave along the keys when that pays (148 SMs assumed)
    assert "whole_units=444 cut_units=68x2" in name(1, 4096, 32, 32, 128, syn.BF16, 4096, idx=False)
    assert "whole_units=444 cut_units=4x8" in name(1, 4096, 28, 4, 128, syn.BF16, 4096, idx=False)
    assert "cut_units=0x1" in name(1, 2048, 32, 32, 128, syn.BF16, 2048, idx=False)
    assert "cut_units=0x1" in name(8, 4096, 32, 32, 128, syn.BF16, 4096, idx=False)
    assert ec.ec_attend_kernel_name(ec.make_desc(1, 64, 4, 4, 64, syn.F32), 65, True, True) == ""   # rejected
