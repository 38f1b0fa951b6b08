"""Host-side checks of the benchmark's bookkeeping: the algorithmic byte / operation model that the
roofline fractions are computed from, and the workload names the command line accepts."""
import os
import sys

import pytest

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402


def mb(x):
    return x / 1e6


def test_algorithmic_bytes_single_linears():
    # 2MK (X) + 2 (MK b_a / 8 + 4M) (codes and r, written then read) + NK/2 + 2NK/G (weights, fp16 scales)
    # + 2MN (Y) + 4N (bias); NVFP4: codes MK/2 + MK/16, weights NK/2 + NK/16 + 4.  Values worked by hand.
    assert mb(bench.algorithmic_bytes_linear(256, 1024, 1024, 64, "w4a8")) == pytest.approx(2.14, abs=0.005)
    assert mb(bench.algorithmic_bytes_linear(1024, 2048, 2048, 16, "nvfp4")) == pytest.approx(13.1, abs=0.05)
    want_2048 = {16: 2.43, 64: 3.02, 128: 3.81, 256: 5.38}
    want_4096 = {16: 9.32, 64: 10.5, 128: 12.1, 256: 15.2}
    want_4096_a4 = {16: 9.26, 64: 10.2, 128: 11.6, 256: 14.2}
    for M in (16, 64, 128, 256):
        assert mb(bench.algorithmic_bytes_linear(M, 2048, 2048, 64, "w4a8")) == pytest.approx(want_2048[M], abs=0.006)
        assert mb(bench.algorithmic_bytes_linear(M, 4096, 4096, 64, "w4a8")) == pytest.approx(want_4096[M], abs=0.06)
        assert mb(bench.algorithmic_bytes_linear(M, 4096, 4096, 64, "w4a4")) == pytest.approx(want_4096_a4[M], abs=0.06)


def test_algorithmic_bytes_and_ops_of_the_blocks():
    c2 = bench.workload_config("cfg2")
    assert c2.ops() / 1e9 == pytest.approx(444.5, abs=0.1)
    assert mb(sum(bench.algorithmic_bytes_linear(c2.M, K, N, 64, "w4a8") for _, K, N in c2.linears)) == pytest.approx(443, abs=1)
    c3 = bench.workload_config("cfg3")
    assert c3.ops() / 1e9 == pytest.approx(3971.8, abs=0.1)
    assert mb(sum(bench.algorithmic_bytes_linear(c3.M, K, N, 64, "w4a4") for _, K, N in c3.linears)) == pytest.approx(2162, abs=1)
    c3f = bench.workload_config("cfg3_nvfp4")
    assert mb(sum(bench.algorithmic_bytes_linear(c3f.M, K, N, 16, "nvfp4") for _, K, N in c3f.linears)) == pytest.approx(2213, abs=1)


@pytest.mark.parametrize("name,scheme,group,suffix", [
    ("cfg2", "w4a8", 64, "m4416"),
    ("cfg2_g128", "w4a8", 128, "_g128"),
    ("cfg2_perchannel", "w4a8", 0, "_per_channel"),
    ("cfg2_perchannel_static", "w4a8", 0, "_per_channel_static"),
    ("cfg3", "w4a4", 64, "m17536"),
    ("cfg3_perchannel", "w4a4", 0, "_per_channel"),
    ("cfg3_nvfp4", "nvfp4", 64, "m17536"),
])
def test_workload_names(name, scheme, group, suffix):
    c = bench.workload_config(name)
    assert c.scheme == scheme and c.group == group and c.name.endswith(suffix)
    assert len(c.linears) == 4 and c.M in (4416, 17536)


def test_unknown_workload_is_refused():
    with pytest.raises(SystemExit):
        bench.workload_config("cfg9")
