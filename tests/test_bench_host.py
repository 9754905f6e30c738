"""Host-side pieces of the benchmark that need no GPU: the DRAM-traffic bookkeeping (a ratio
measured on other kernel sources must not be reported) and the ncu csv reader."""
import os

from paper_2607_24260_b200 import traffic


def test_traffic_ratio_is_dropped_when_the_kernel_sources_changed(tmp_path, monkeypatch):
    f = tmp_path / "traffic_ratio.txt"
    monkeypatch.setattr(traffic, "RATIO_FILE", str(f))
    assert traffic.read_ratios() == {"decode": None, "verify": None}          # no file
    traffic.write_ratio("decode", 1.0278, "note")
    traffic.write_ratio("verify", 1.0032, "note")
    traffic.write_ratio("decode", 1.03, "second capture replaces the first")
    got = traffic.read_ratios()
    assert got == {"decode": 1.03, "verify": 1.0032}
    # the same file read against other sources: nothing is reported
    monkeypatch.setattr(traffic, "kernel_digest", lambda: "0" * 16)
    assert traffic.read_ratios() == {"decode": None, "verify": None}


def test_tracked_ratio_file_parses_and_is_plausible():
    """profiles/traffic_ratio.txt as committed: two entries, ratios of a kernel that reads every
    byte once (1.00 .. 1.05), written for a 16-hex-digit digest."""
    rows = [l.split() for l in open(traffic.RATIO_FILE) if l.strip() and not l.startswith("#")]
    kinds = {r[0]: r for r in rows}
    assert set(kinds) == {"decode", "verify"}
    for r in rows:
        assert 1.0 <= float(r[1]) <= 1.05 and len(r[2]) == 16 and int(r[2], 16) >= 0


def test_ncu_csv_reader(tmp_path):
    csv_text = (
        '"ID","Kernel Name","Grid Size","dram__bytes_read.sum","dram__bytes_write.sum","x"\n'
        '"","","","Mbyte","Kbyte",""\n'
        '"0","void kap::kap_attn_split_kernel<1, 0>(CUtensorMap_st, kap::AttnParams)","(320, 1, 1)","117.5","3,000","1"\n'
        '"1","void kap::kap_attn_split_kernel<2, 0>(CUtensorMap_st, kap::AttnParams)","(440, 1, 1)","2147.8","6,500","1"\n'
        '"2","other_kernel","(1, 1, 1)","9","9","1"\n')
    p = tmp_path / "raw.csv"
    p.write_text(csv_text)
    assert abs(traffic.traffic_from_csv(str(p), "split_kernel<1") - (117.5e6 + 3.0e6)) < 1
    assert abs(traffic.traffic_from_csv(str(p), "split_kernel<2") - (2147.8e6 + 6.5e6)) < 1
    both = traffic.traffic_from_csv(str(p))
    assert abs(both - (117.5e6 + 3.0e6 + 2147.8e6 + 6.5e6) / 2) < 1
