"""Host-side helpers of bench.py: the roofline arithmetic and the rule that the DRAM-traffic figure is only reported for
the kernel source it was captured on."""
import hashlib
import os
import re

import bench
from paper_2506_10848_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_step_flops_and_bytes_at_the_8b_shape():
    g, a, h = bench.step_flops(W.LLADA_8B, 512, 512, 256)
    assert abs(g - 7.147e12) / 7.147e12 < 2e-3            # 436.2 MFLOP per token and layer
    assert abs(a - 4.0 * 512 * 512 * 4096 * 32) < 1 and abs(h - 2.0 * 256 * 4096 * 126464) < 1
    by = bench.step_bytes(W.LLADA_8B, 512, 256)
    assert 16.5e9 < by < 18.5e9                              # 15 GB of weights + activations + logits


def test_traffic_is_reported_only_for_the_captured_kernel_source(tmp_path, monkeypatch):
    path = os.path.join(ROOT, "profiles", "gemm_kernel_llada8b_dram_traffic.md")
    text = open(path).read()
    sha = hashlib.sha256(open(os.path.join(ROOT, "paper_2506_10848_b200", "csrc", "gemm_tcgen05.cu"), "rb").read()).hexdigest()
    recorded = re.search(r"kernel_source_sha256:\s*([0-9a-f]{64})", text).group(1)
    got = bench.gemm_traffic_from_profiles()
    if recorded == sha:
        assert got is not None and 1.0e8 < got < 1.6e8      # about the 116 MB of weights a launch streams
    else:
        assert got is None                                   # the kernel changed since the capture: no stale figure
    # a copy of the repository layout whose summary carries another hash must give None
    fake = tmp_path / "r"
    (fake / "profiles").mkdir(parents=True)
    (fake / "paper_2506_10848_b200" / "csrc").mkdir(parents=True)
    (fake / "profiles" / "gemm_kernel_llada8b_dram_traffic.md").write_text("traffic_bytes_per_launch: 123\nkernel_source_sha256: " + "0" * 64 + "\n")
    (fake / "paper_2506_10848_b200" / "csrc" / "gemm_tcgen05.cu").write_text("// another kernel\n")
    monkeypatch.setattr(bench, "ROOT", str(fake))
    assert bench.gemm_traffic_from_profiles() is None
    good = hashlib.sha256(b"// another kernel\n").hexdigest()
    (fake / "profiles" / "gemm_kernel_llada8b_dram_traffic.md").write_text("traffic_bytes_per_launch: 123\nkernel_source_sha256: " + good + "\n")
    assert bench.gemm_traffic_from_profiles() == 123.0
