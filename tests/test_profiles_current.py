"""The ncu summaries under profiles/ that bench.py reads its `roofline.traffic` figures from are stamped with a hash of
the kernel sources they were captured on; a stale stamp makes the bench line say `traffic: null`."""
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402


def test_traffic_profiles_match_the_kernel_sources():
    for name in bench.TRAFFIC_PROFILES:
        value, where = bench.ncu_traffic(name, launch_bytes=1.0e8)
        assert value is not None and value > 0, f"{name}: {where}"


def test_every_profile_summary_names_its_command():
    root = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "profiles")
    for f in sorted(os.listdir(root)):
        assert f.endswith((".md", ".txt")), f
        text = open(os.path.join(root, f)).read()
        assert "python " in text or "ncu " in text, f"{f}: no command"
        assert len(text) < 16384, f"{f}: keep summaries short"
