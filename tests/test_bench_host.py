"""Host-side pieces of bench.py that need no GPU: the bounded oracle sample of the CPU
baseline and reference arm, the byte count both arms share, and the stamped DRAM-traffic file."""
import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench
import oracle
from paper_1606_07676_b200 import binding as iso
from paper_1606_07676_b200 import workloads as wl
from schedule_sim import make_request


def test_oracle_sample_equals_the_oracle_on_the_whole_workload():
    """The sample reserves the host send buffer in full and generates only the planes its ranks
    read from (here across the wrap-around); what the oracle computes on it must be what it
    computes on the whole buffer."""
    w = wl.Workload("s", "alltoall", (16, 12, 5), wl.moore(3, 2), 24, kind="uint8", seed=5)
    whole = bench.OracleSample(w)                          # small: taken whole
    assert (whole.r0, whole.r1) == (0, w.P)
    part = bench.OracleSample(w, max_out_bytes=3 * 60 * whole.rs, whole_below=0)    # 3 of 16 planes of 60 processes
    assert (part.r0, part.r1) == (0, 180) and "7 source planes" in part.what       # planes 14, 15, 0..4
    assert np.array_equal(part.run(), whole.run()[:180])
    assert part.bytes_min * w.P == whole.bytes_min * 180 and part.nominal_moved() * w.P == whole.nominal_moved() * 180
    for kind in ("allgather", "alltoallv"):
        lens = np.array([1 + 7 * i for i in range(len(w.offsets))]) if kind == "alltoallv" else None
        w2 = wl.Workload("s", kind, w.dims, w.offsets, 24, lens=lens, kind="uint8", seed=7)
        a, b = bench.OracleSample(w2), bench.OracleSample(w2, max_out_bytes=2 * 60 * wl.layout(w2)[4], whole_below=0)
        assert b.r1 == 120 and np.array_equal(b.run(), a.run()[:120]), kind


@pytest.mark.parametrize("name", ["cfg1", "cfg2_alltoall", "cfg2_allgather", "cfg3_m64", "cfg3_m4096", "cfg4", "cfg5",
                                  "octant_d3r3_alltoall", "shells_d3_alltoall"])
def test_both_arms_count_the_same_bytes(name):
    """The reference arm takes its byte count from the paper's formula (oracle/counters.py: a
    block hops once per non-zero coordinate), the GPU arm from the library's statistics; for the
    driver's ratio to be a ratio of times they must be the same number."""
    w = wl.config(name)
    comm, req = make_request(w)
    iso.Iso_request_set_sender_side(req, 0)                # the receiver-side count: one read per copy
    st = iso.Iso_request_get_stats(req)
    iso.Iso_request_free(req)
    iso.Iso_comm_free(comm)
    sample = bench.OracleSample.__new__(bench.OracleSample)
    sample.w = w
    sample.lens, sample.sd, sample.rd, sample.ss, sample.rs = wl.layout(w)
    sample.ranks = w.P
    assert sample.nominal_moved() == st["bytes_moved"]
    assert 2 * w.P * int(sample.lens.sum()) == st["bytes_min"]


def test_config_object_is_the_same_in_both_arms():
    w = wl.config(bench.HEADLINE)
    a, b = bench.config_dict(w, 1, 1), bench.config_dict(w, 1, 1)
    assert a == b and a["workload"] == "cfg3_m4096" and "model" not in a
    assert bench.replica_count(w) == 1 and bench.replica_count(wl.config("cfg2_alltoall")) == 5


def test_traffic_entries_are_ignored_once_the_kernels_change(tmp_path, monkeypatch):
    now = bench.sources_hash()
    f = tmp_path / "dram_traffic.txt"
    f.write_text("# comment\n"
                 "cfg3_m4096 combining 2 20626400000 cold x8 %s abc\n"
                 "cfg2_alltoall combining 3 174292000 warm as_is 0000000000000000 abc\n" % now)
    monkeypatch.setattr(bench, "TRAFFIC_FILE", str(f))
    got = bench.recorded_traffic("cfg3_m4096", "combining")
    assert got and got["bytes_per_step"] == 20626400000.0 and got["launches"] == 2
    assert bench.recorded_traffic("cfg2_alltoall", "combining") is None      # stamped with other sources
    assert bench.recorded_traffic("cfg3_m4096", "direct") is None
    # the tracked file is well formed: workload, schedule, launches, bytes, mode, scaling, 16-hex stamp, commit
    monkeypatch.undo()
    rows = [ln.split() for ln in open(bench.TRAFFIC_FILE) if ln.strip() and not ln.startswith("#")]
    assert rows and all(len(f) == 8 and int(f[2]) > 0 and float(f[3]) > 0 and len(f[6]) == 16 for f in rows)
    assert any(f[0] == bench.HEADLINE and f[1] == "combining" for f in rows)
