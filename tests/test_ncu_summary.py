"""The ncu CSV summariser behind profiles/: parsing, per-kernel aggregation and the traffic record
(host only; the CSV below has the layout `ncu --csv --log-file` writes)."""
import os

from paper_2501_07161_b200 import ncu_summary as N

CSV = '''==PROF== Connected to process 1
"ID","Process ID","Process Name","Host Name","Kernel Name","Context","Stream","Block Size","Grid Size","Device","CC","Section Name","Metric Name","Metric Unit","Metric Value"
"0","1","python","h","void qv2::<unnamed>::metrics_kernel<0, 0, 0>(qv2::MetricsArgs)","1","7","(256, 1, 1)","(444, 1, 1)","0","10.0","Command line profiler metrics","dram__bytes_read.sum","Mbyte","987.94"
"0","1","python","h","void qv2::<unnamed>::metrics_kernel<0, 0, 0>(qv2::MetricsArgs)","1","7","(256, 1, 1)","(444, 1, 1)","0","10.0","Command line profiler metrics","dram__bytes_write.sum","Kbyte","360.00"
"0","1","python","h","void qv2::<unnamed>::metrics_kernel<0, 0, 0>(qv2::MetricsArgs)","1","7","(256, 1, 1)","(444, 1, 1)","0","10.0","Command line profiler metrics","gpu__time_duration.sum","us","162.95"
"1","1","python","h","qv2::<unnamed>::rank_kernel(unsigned int)","1","7","(256, 1, 1)","(1, 1, 1)","0","10.0","Command line profiler metrics","dram__bytes_read.sum","Kbyte","50.00"
"1","1","python","h","qv2::<unnamed>::rank_kernel(unsigned int)","1","7","(256, 1, 1)","(1, 1, 1)","0","10.0","Command line profiler metrics","dram__bytes_write.sum","byte","0"
"1","1","python","h","qv2::<unnamed>::rank_kernel(unsigned int)","1","7","(256, 1, 1)","(1, 1, 1)","0","10.0","Command line profiler metrics","gpu__time_duration.sum","ns","10300"
"2","1","python","h","void qv2::<unnamed>::metrics_kernel<0, 0, 0>(qv2::MetricsArgs)","1","7","(256, 1, 1)","(444, 1, 1)","0","10.0","Command line profiler metrics","dram__bytes_read.sum","Gbyte","0.98794"
"2","1","python","h","void qv2::<unnamed>::metrics_kernel<0, 0, 0>(qv2::MetricsArgs)","1","7","(256, 1, 1)","(444, 1, 1)","0","10.0","Command line profiler metrics","dram__bytes_write.sum","Kbyte","360.00"
"2","1","python","h","void qv2::<unnamed>::metrics_kernel<0, 0, 0>(qv2::MetricsArgs)","1","7","(256, 1, 1)","(444, 1, 1)","0","10.0","Command line profiler metrics","gpu__time_duration.sum","ms","0.16305"
'''


def test_launch_list_units_and_aggregation(tmp_path):
    p = tmp_path / "l.csv"
    p.write_text(CSV)
    launches = N.read_launch_list(str(p))
    assert list(launches) == ["0", "1", "2"]
    assert abs(launches["1"]["gpu__time_duration.sum"] - 10.3) < 1e-9          # ns -> us
    assert abs(launches["2"]["gpu__time_duration.sum"] - 163.05) < 1e-9         # ms -> us
    assert abs(launches["2"]["dram__bytes_read.sum"] - 987.94e6) < 1.0          # Gbyte -> byte
    agg = N.by_kernel(launches)
    (mk, m), (rk, r) = list(agg.items())
    assert "metrics_kernel<0, 0, 0>" in mk and m["launches"] == 2 and r["launches"] == 1
    text = N.cmd_launches(str(p))
    assert "launches=   2" in text and "share=" in text and "dram_read_MB/launch=" in text
    assert text.splitlines()[0].startswith("qv2::<") or "metrics_kernel" in text.splitlines()[0]   # sorted by time


def test_traffic_record_round_trips_through_bench(tmp_path):
    p = tmp_path / "l.csv"
    p.write_text(CSV)
    out = tmp_path / "traffic.txt"
    N.cmd_traffic(str(p), "metrics_kernel", 987210496, str(out), "test")
    rec = dict(ln.split(":", 1) for ln in out.read_text().splitlines() if ":" in ln and not ln.startswith("#"))
    assert abs(float(rec["dram_bytes_per_algorithmic_byte"]) - (987.94e6 + 360e3) / 987210496) < 1e-5
    assert rec["sha256"].strip() == N.sources_hash()
    for rel in rec["sources"].split():
        assert os.path.exists(os.path.join(N.ROOT, rel))
