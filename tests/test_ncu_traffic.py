"""Host logic of the DRAM-traffic record: parsing both CSV layouts ncu writes, and the staleness rule
(a record is only returned while the kernel's source file is the one the counters were taken from)."""
import json
import os

from paper_2603_14303_b200 import ncu_traffic

RAW = '''"ID","Process ID","Kernel Name","dram__bytes_read.sum","dram__bytes_write.sum","gpu__time_duration.sum"
"","","","Mbyte","Kbyte","us"
"0","1","void other_kernel(int)","1.0","1.0","3.0"
"1","1","dm::decode_mma_kernel(const __nv_bfloat16 *, int)","34.5","100.0","17.0"
"2","1","dm::decode_mma_kernel(const __nv_bfloat16 *, int)","33.5","300.0","17.0"
'''

LONG = '''==PROF== noise line
"ID","Process ID","Process Name","Kernel Name","Metric Name","Metric Unit","Metric Value"
"0","1","python","cf::compress_fused_kernel<2>(Params)","dram__bytes_read.sum","byte","1,000"
"0","1","python","cf::compress_fused_kernel<2>(Params)","dram__bytes_write.sum","byte","500"
"0","1","python","cf::compress_fused_kernel<2>(Params)","gpu__time_duration.sum","us","70"
"1","1","python","other(int)","dram__bytes_read.sum","byte","7"
'''


def test_both_csv_layouts(tmp_path):
    raw, long_ = tmp_path / "raw.csv", tmp_path / "long.csv"
    raw.write_text(RAW)
    long_.write_text(LONG)
    got = ncu_traffic.parse_ncu_csv(str(raw), "decode_mma_kernel")
    assert got == [(34.5e6, 100e3), (33.5e6, 300e3)]
    assert ncu_traffic.parse_ncu_csv(str(long_), "compress_fused") == [(1000.0, 500.0)]
    assert ncu_traffic.parse_ncu_csv(str(long_), "decode_mma") == []


def test_record_goes_stale_when_the_kernel_source_changes(tmp_path, monkeypatch):
    rec = tmp_path / "traffic.txt"
    monkeypatch.setattr(ncu_traffic, "RECORD", str(rec))
    good = ncu_traffic.source_hash("decode")
    assert good is not None and len(good) == 16
    rec.write_text(json.dumps({
        "w/decode": {"dram_bytes_per_launch": 123.0, "source_sha256_16": good},
        "w/compress": {"dram_bytes_per_launch": 456.0, "source_sha256_16": "0" * 16}}))
    assert ncu_traffic.lookup("w", "decode") == 123.0
    assert ncu_traffic.lookup("w", "compress") is None          # counters of a kernel that has changed since
    assert ncu_traffic.lookup("other", "decode") is None
    os.remove(rec)
    assert ncu_traffic.lookup("w", "decode") is None
