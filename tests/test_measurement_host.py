"""Host logic of the measurement path (no GPU): the launch-list summary, and the rule that DRAM traffic
figures are only reported for the kernel sources they were measured on."""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2002_11082_b200 import profile_summary  # noqa: E402


def test_launch_list_summary_shares(tmp_path):
    log = tmp_path / "launches.csv"
    rows = ['"ID","Process ID","Process Name","Host Name","Kernel Name","Context","Stream","Block Size","Grid Size",'
            '"Device","CC","Section Name","Metric Name","Metric Unit","Metric Value"']
    times = [("ogq::k_sel_round1(ogq::SelArgs)", 200.0), ("ogq::k_sel_round2(ogq::SelArgs)", 300.0),
             ("ogq::k_sel_round1(ogq::SelArgs)", 100.0), ("void ogq::k_quantize_pack<4, 0, 0>(float const*)", 400.0)]
    for i, (name, us) in enumerate(times):
        rows.append(f'"{i}","1","python","host","{name}","1","7","(512, 1, 1)","(296, 1, 1)","0","10.0",'
                    f'"Command line profiler metrics","gpu__time_duration.sum","us","{us}"')
    log.write_text("==PROF== connected\n" + "\n".join(rows) + "\n")
    out = tmp_path / "out.md"
    profile_summary.cmd_launches([str(out), str(log)])
    text = out.read_text().splitlines()
    assert text[0].startswith("| kernel | launches |")
    body = {ln.split("|")[1].strip(): [c.strip() for c in ln.split("|")[2:-1]] for ln in text[2:]}
    assert body["k_quantize_pack<4, 0, 0>"] == ["1", "400.0", "400.0", "0.400"]
    assert body["k_sel_round1"] == ["2", "300.0", "150.0", "0.300"]
    assert body["k_sel_round2"] == ["1", "300.0", "300.0", "0.300"]
    # largest total first
    assert text[2].split("|")[1].strip() == "k_quantize_pack<4, 0, 0>"


def test_unit_scaling_of_report_values():
    assert profile_summary._to_number("1,500", "ns") == 1.5          # times in microseconds
    assert profile_summary._to_number("2", "ms") == 2000.0
    assert profile_summary._to_number("3", "Gbyte") == 3000.0        # bytes in MB
    assert profile_summary._to_number("4,096", "Kbyte") == 4.096
    assert profile_summary._to_number("7", "") == 7.0


def test_traffic_only_for_the_sources_it_was_measured_on(monkeypatch):
    import bench

    path = os.path.join(ROOT, "profiles", "dram_bytes_per_element.json")
    rec = json.load(open(path))
    h = profile_summary.kernel_sources_hash()
    assert len(h) == 64 and h == profile_summary.kernel_sources_hash()  # a sha256, stable
    assert bench.kernel_sources_hash() == h                             # bench hashes the same files
    key = next(iter(rec["entries"]))
    kernel, scheme = key.split("|")
    monkeypatch.setattr(bench, "kernel_sources_hash", lambda: rec["sources_sha256"])
    assert bench.stored_traffic(kernel, scheme) == rec["entries"][key]
    assert bench.stored_traffic("k_no_such_kernel", scheme) is None
    monkeypatch.setattr(bench, "kernel_sources_hash", lambda: "0" * 64)  # the sources changed since
    assert bench.stored_traffic(kernel, scheme) is None
