"""Host-side logic of bench.py that needs no GPU: where the roofline's `traffic` comes from, the algorithmic byte
and flop counts, and the whole-job throughput formula."""
import os
import re
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
import mdn_workloads as wl  # noqa: E402


def test_traffic_is_read_from_the_committed_ncu_summaries():
    """`roofline.traffic` is not a typed-in constant: it is the `traffic_bytes_per_launch` line of the ncu summary of
    exactly the kernel and workload being timed, and null for anything else."""
    for stage, fname in bench.PROFILE_FILES.items():
        text = open(os.path.join(ROOT, "profiles", fname)).read()
        fields = dict(re.findall(r"^(kernel|workload|traffic_bytes_per_launch)\s*=\s*(\S+)\s*$", text, flags=re.M))
        assert fields["kernel"] == bench.STAGE_KERNELS[stage] and fields["workload"] == wl.CONFIGS[2].name
        got, src = bench.profile_traffic(stage, wl.CONFIGS[2].name)
        assert got == float(fields["traffic_bytes_per_launch"]) and src["file"] == "profiles/" + fname
        # the number the summary's table shows (MB, read + write) is the same number
        mb = float(fields["traffic_bytes_per_launch"]) / 1e6
        assert ("%.1f MB" % mb) in text
        assert bench.profile_traffic(stage, wl.CONFIGS[1].name)[0] is None          # another workload: no number
    assert bench.profile_traffic("coeff_scan", wl.CONFIGS[2].name)[0] is None        # a stage with no summary


def test_algorithmic_bytes_and_flops_of_the_headline_workload():
    w = wl.CONFIGS[2]
    per_head_token = 2 * (2 * w.dk + 2 * w.dv) + 16          # bf16 q, k, v in, o out, four fp32 gates
    assert per_head_token == 1040
    states = 2 * w.B * w.H * w.dk * w.dv * 4                 # final S and M
    assert bench.algorithmic_bytes(w, w.B, False) == w.B * w.T * w.H * per_head_token + states
    assert bench.algorithmic_flops(w) == w.B * w.T * w.H * (12 * w.dk * w.dv + 4 * 64 * (w.dk + w.dv))
    assert abs(bench.algorithmic_bytes(w, w.B, False) - 562.0e6) < 0.1e6


def test_whole_job_throughput():
    w = wl.CONFIGS[2]
    assert bench.job_tokens_per_s(w, 1, 10, 4.0) == w.B * w.T * 10 / 4.0e-3
    assert bench.job_tokens_per_s(w, 8, 10, 4.0) == 8 * bench.job_tokens_per_s(w, 1, 10, 4.0)
