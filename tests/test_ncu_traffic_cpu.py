"""The store of measured DRAM traffic that bench.py reports: a capture is parsed by kernel, kept with
the digest of the kernel sources, and withheld as soon as the sources no longer have that digest."""
import json

from paper_2605_08632_b200 import ncu_traffic as N

HDR = '"ID","Process ID","Process Name","Host Name","Kernel Name","Context","Stream","Block Size","Grid Size","Device","CC","Section Name","Metric Name","Metric Unit","Metric Value"'


def _row(i, kernel, metric, value):
    return f'"{i}","1","python","h","void {kernel}(CUtensorMap_st, Sched, int *)","1","7","(192, 1, 1)","(148, 1, 1)","0","10.0","Command line profiler metrics","{metric}","byte","{value}"'


def test_record_load_and_invalidation(tmp_path, monkeypatch):
    kernels = ["gemm_kernel<0, 0, EpiFwdT<2>, 2>", "gemm_kernel<0, 1, EpiOut, 2>", "gemm_kernel<1, 1, EpiOut, 2>", "other_kernel<1>"]
    lines = ["==PROF== Connected", HDR]
    for step in range(2):
        for j, k in enumerate(kernels):
            i = step * 4 + j
            lines += [_row(i, k, "dram__bytes_read.sum", 1000 * (i + 1)), _row(i, k, "dram__bytes_write.sum", "1,0" + str(i)),
                      _row(i, k, "gpu__time_duration.sum", 5)]
    csv_path = tmp_path / "cap.csv"
    csv_path.write_text("\n".join(lines) + "\n")
    monkeypatch.setattr(N, "STORE", str(tmp_path / "store.json"))
    ent = N.record(str(csv_path), "config2", 16384, "fused")
    assert set(ent["stages"]) == {"logits", "dH", "dW"} and len(ent["stages"]["dH"]) == 2
    got = N.load("config2", 16384, "fused")
    assert N.bytes_of(got, "dH", 0, 1) == 6000 + 105            # the last captured step: launch ID 5
    assert N.bytes_of(got, "dH", 1, 1) is None and N.bytes_of(got, "fwd_two_call", 0, 1) is None
    assert N.load("config2", 8192, "fused") is None and N.load("config3", 16384, "fused") is None
    # a changed kernel source invalidates the numbers
    store = json.load(open(N.STORE))
    store["config2:16384:fused"]["source_digest"] = "0" * 64
    json.dump(store, open(N.STORE, "w"))
    assert N.load("config2", 16384, "fused") is None


def test_committed_store_is_well_formed():
    import os
    if os.path.exists(N.STORE):
        for key, ent in json.load(open(N.STORE)).items():
            assert len(key.split(":")) == 3 and len(ent["source_digest"]) == 64
            for launches in ent["stages"].values():
                assert all(l["read"] >= 0 and l["write"] >= 0 for l in launches)
