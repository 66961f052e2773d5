"""bench.py turns measured times into roofline fractions with per-env-step instruction counts
that come from profiler captures. The captures are only valid for the kernel sources they were
taken from: this test fails when those sources have changed since (re-capture, update the
constants and the summaries under profiles/, then record the new hash)."""
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_instruction_counts_belong_to_the_current_kernel_sources():
    import bench
    from paper_2301_13062_b200 import build
    assert bench.COUNTED_AT == build.kernel_hash(), (
        "the rollout / step kernel sources changed after the instruction counts in bench.py were captured")


def test_profile_summaries_name_the_same_sources():
    import bench
    named = set()
    for name in os.listdir(os.path.join(ROOT, "profiles")):
        text = open(os.path.join(ROOT, "profiles", name)).read()
        named.update(re.findall(r"kernel sources at `([0-9a-f]{16})`", text))
    assert bench.COUNTED_AT in named, "no summary under profiles/ was captured from the sources bench.py counts on"
    for variant, ops in bench.ROLLOUT_OPS.items():
        assert ops["thread"] > 0 and ops["slot"] > 0 and ops["kernel"].startswith("rollout_")
