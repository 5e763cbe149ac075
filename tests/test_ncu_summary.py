"""The ncu CSV reader that writes the summaries under profiles/: launch list shares and the DRAM-bytes table."""
from paper_2209_05433_b200 import ncu_summary

LAUNCHES = '''==PROF== Connected to process 1
"ID","Process ID","Process Name","Host Name","Kernel Name","Context","Stream","Block Size","Grid Size","Device","CC","Section Name","Metric Name","Metric Unit","Metric Value"
"0","1","python","box","void fp8b200::gemm::k_gemm_fp8<2, 1, 8, 1>(CUtensorMap_st, int)","1","7","(384, 1, 1)","(148, 1, 1)","0","10.0","Command line profiler metrics","gpu__time_duration.sum","msecond","3.0"
"1","1","python","box","void fp8b200::k_amax<1, 8>(const void *, unsigned long)","1","7","(256, 1, 1)","(9000, 1, 1)","0","10.0","Command line profiler metrics","gpu__time_duration.sum","usecond","250"
"2","1","python","box","void fp8b200::k_amax<1, 8>(const void *, unsigned long)","1","7","(256, 1, 1)","(9000, 1, 1)","0","10.0","Command line profiler metrics","gpu__time_duration.sum","usecond","750"
'''

RAW = '''"ID","Kernel Name","dram__bytes_read.sum","dram__bytes_write.sum","gpu__time_duration.sum"
"","","Gbyte","Mbyte","msecond"
"0","void fp8b200::gemm::k_gemm_fp8<2, 1, 8, 1>(CUtensorMap_st, int)","3.0","800","3.4"
"1","void fp8b200::gemm::k_gemm_fp8<2, 1, 8, 1>(CUtensorMap_st, int)","3.2","800","3.4"
"2","void fp8b200::k_amax<1, 8>(const void *, unsigned long)","1.2","0","0.2"
'''


def test_launch_list_counts_times_and_shares(tmp_path):
    f = tmp_path / "launches.csv"
    f.write_text(LAUNCHES)
    text = ncu_summary.launch_list(ncu_summary._rows(str(f)))
    lines = text.splitlines()
    assert lines[1].split() == ["1", "3000.0", "75.00%", "k_gemm_fp8<2,", "1,", "8,", "1>"]
    assert lines[2].split()[:3] == ["2", "1000.0", "25.00%"] and "k_amax<1, 8>" in lines[2]


def test_raw_page_rewrites_one_line_of_the_traffic_table(tmp_path, monkeypatch):
    f = tmp_path / "raw.csv"
    f.write_text(RAW)
    table = tmp_path / "dram_traffic.txt"
    table.write_text("other.kernel 1.000000e+09   # kept\nk_gemm.test 9.9e+09   # replaced\n")
    monkeypatch.setattr(ncu_summary, "TRAFFIC_FILE", str(table))
    monkeypatch.setattr(ncu_summary, "ROOT", str(tmp_path))
    text = ncu_summary.raw_page(ncu_summary._rows(str(f)), "k_gemm_fp8", "k_gemm.test")
    assert text.count("--- k_gemm_fp8<2, 1, 8, 1>") == 2 and "k_amax" not in text
    lines = table.read_text().splitlines()
    assert lines[0].startswith("other.kernel 1.000000e+09")
    name, value = lines[1].split()[:2]
    assert name == "k_gemm.test" and abs(float(value) - 3.9e9) < 1e3          # mean of (3.0 + 0.8) and (3.2 + 0.8) GB
    assert len(lines) == 2
