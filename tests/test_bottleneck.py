"""The three-way classification rule of the paper's Table 2 (thresholds at 30 %)."""
from paper_2603_07169_b200 import bottleneck as bn


def test_rule_of_table_2():
    assert bn.classify(45.0, 10.0, 10.0) == "compute"          # compute above 30 % wins whatever memory does
    assert bn.classify(45.0, 90.0, 90.0) == "compute"
    assert bn.classify(10.0, 10.0, 10.0) == "latency"          # everything idle: waiting on memory latency
    assert bn.classify(10.0, 29.9, 29.9) == "latency"
    assert bn.classify(10.0, 80.0, 10.0) == "bandwidth"        # either memory throughput above 30 %
    assert bn.classify(10.0, 10.0, 80.0) == "bandwidth"
    assert bn.classify(30.0, 30.0, 30.0) == "bandwidth"        # the default class at the boundary


def test_csv_post_processing():
    header = ["ID", "Kernel Name", bn.COMPUTE_TH, bn.DRAM_TH, bn.MEMORY_TH, "lts__t_sector_hit_rate.pct", "l1tex__t_sector_hit_rate.pct"]
    units = ["", "", "%", "%", "%", "%", "%"]
    rows = [header, units, ["0", "k_stream", "7.4", "83.0", "83.0", "6.0", "80.0"], ["1", "k_tiny", "7.0", "3.0", "4.0", "9.6", "38.1"],
            ["2", "k_fma", "61.0", "5.0", "20.0", "50", "50"]]
    recs = bn.classify_rows(rows)
    assert [r["class"] for r in recs] == ["bandwidth", "latency", "compute"]
    assert recs[1]["filtered"]["lts__t_sector_hit_rate.pct"] == 9.6
    assert set(recs[0]["filtered"]) == set(bn.FILTERED["bandwidth"])
