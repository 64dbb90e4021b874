"""The bench's last stdout line is what a harness parses: it must stay short and complete."""
import io
import json
from contextlib import redirect_stdout

import bench

REQUIRED = ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
            "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline")


def _stub_headline():
    roofline = {"bound": "hbm", "kernel": "scan_kernel<4,1,1,256,16,4> (retrace)", "achieved": 6241.123, "peak": 6530.3,
                "unit": "GB/s", "frac": 0.9557, "traffic": 738443008, "algorithmic_bytes_per_launch": 743445888,
                "peak_source": "of measured", "all_kernels_frac": 0.9512}
    e2e = {"value": 9543211234.123456, "unit": bench.METRIC, "h2d_bytes_per_step": 1040252928, "d2h_bytes_per_step": 1207959552,
           "steps": 8, "ms_per_step": 24.6123, "note": "pinned host -> device, seven C-ABI calls, all outputs -> pinned host; three streams"}
    cpu = {"value": 405976369.8539816, "unit": bench.METRIC, "cores": 128, "kind": "oracle",
           "sample": "first 16384 of 16384 rows x T=2048, all seven algorithms once, 19.87 s, fp64 sequential C oracle, rows split "
                     "over 128 host threads (single thread: first 1024 rows, 3.21 s)"}
    clocks = {"sm_mhz": 1965, "sm_max_mhz": 1965, "reasons": ["sw_power_cap", "sw_thermal_slowdown"], "samples": 12345,
              "power_w_max": 1000.0}
    small = {f"{a}_{t}{s}": 0.123 for a in ("gae", "vtr") for t in (256, 512, 1024) for s in ("", "t")}
    small.update({"gae_16384": 0.412, "disc_16384": 0.293})
    workload = ("config 5: all seven algorithms, num_envs=16384, T=2048, fp32, dones~Bern(0.02), truncs~Bern(0.005) "
                "with per-step truncation handling, gamma=0.99, lambda=0.95; 7 launches per step")
    return bench.build_headline(value=413123456789.123, world=8, steps=200, warmup=5, ms_per_step=0.56912, workload=workload,
                                clocks=clocks, e2e=e2e, launches=1400, roofline=roofline, cpu_baseline=cpu,
                                per_algorithm_frac={a: 0.9876 for a in bench.ALGOS}, small_frac=small,
                                detail_file="out/bench_detail.json")


def test_headline_is_short_and_complete():
    h = _stub_headline()
    text = json.dumps(h)
    assert len(text) < bench.HEADLINE_LIMIT, len(text)
    for k in REQUIRED:
        assert k in h, k
    for k in ("achieved", "peak", "frac", "traffic", "bound", "unit"):
        assert k in h["roofline"]
    for k in ("value", "unit", "h2d_bytes_per_step", "d2h_bytes_per_step"):
        assert k in h["e2e"]
    for k in ("value", "unit", "cores", "kind", "sample"):
        assert k in h["cpu_baseline"]
    assert "workload" in h["config"] and "model" not in h["config"]


def test_headline_is_the_last_line_printed():
    details = [{"detail": "sweep", "blob": "x" * 5000}, {"detail": "per_algorithm", "per_algorithm": {"gae": {"ms": 0.1}}}]
    buf = io.StringIO()
    with redirect_stdout(buf):
        bench.emit(details, _stub_headline())
    lines = buf.getvalue().strip().split("\n")
    assert len(lines) == len(details) + 1
    last = json.loads(lines[-1])
    assert last["metric"] == bench.METRIC and last["value"] > 0 and "roofline" in last
    assert len(lines[-1]) < bench.HEADLINE_LIMIT
    assert all("detail" in json.loads(ln) for ln in lines[:-1])


def test_oversized_headline_sheds_optional_keys_first():
    h = _stub_headline()
    h["small_configs_frac_of_peak"] = {f"k{i}": 0.5 for i in range(400)}
    buf = io.StringIO()
    with redirect_stdout(buf):
        bench.emit([], h)
    last = json.loads(buf.getvalue().strip().split("\n")[-1])
    assert "small_configs_frac_of_peak" not in last and "roofline" in last and "cpu_baseline" in last


def test_traffic_is_null_for_another_kernel_instance():
    table = {"retrace": {"kernel": "scan_kernel<4,1,1,256,8,4>", "dram_bytes_per_launch": 738443008}}
    assert bench.traffic_for("retrace", "scan_kernel<4,1,1,256,8,4>", table) == 738443008
    assert bench.traffic_for("retrace", "scan_kernel<4,1,1,128,16,5>", table) is None
    assert bench.traffic_for("gae", "scan_kernel<0,1,1,128,16,6>", table) is None


def test_traffic_table_from_an_ncu_log(tmp_path):
    log = tmp_path / "dram.csv"
    log.write_text(
        '==PROF== Connected to process 1\n'
        '"ID","Process ID","Process Name","Host Name","Kernel Name","Context","Stream","Block Size","Grid Size","Device","CC",'
        '"Section Name","Metric Name","Metric Unit","Metric Value"\n'
        '"0","1","python","h","void scan_kernel<4, 1, 1, 256, 8, 4, 0>(ScanParams)","1","7","(256, 1, 1)","(16384, 1, 1)","0","10.0",'
        '"Command line profiler metrics","dram__bytes_read.sum","Mbyte","623.6"\n'
        '"0","1","python","h","void scan_kernel<4, 1, 1, 256, 8, 4, 0>(ScanParams)","1","7","(256, 1, 1)","(16384, 1, 1)","0","10.0",'
        '"Command line profiler metrics","dram__bytes_write.sum","Mbyte","114.8"\n'
        '"1","1","python","h","void rlcs::scan_kernel<0, true, true, 128, 16, 6, false>(rlcs::ScanParams)","1","7","(128, 1, 1)","(16384, 1, 1)","0","10.0",'
        '"Command line profiler metrics","dram__bytes_read.sum","byte","1,000"\n'
        '"1","1","python","h","void rlcs::scan_kernel<0, true, true, 128, 16, 6, false>(rlcs::ScanParams)","1","7","(128, 1, 1)","(16384, 1, 1)","0","10.0",'
        '"Command line profiler metrics","dram__bytes_write.sum","byte","24"\n')
    out = tmp_path / "t.json"
    doc = bench.traffic_from_ncu(str(log), out_path=str(out), command="ncu ...")
    assert doc["kernels"]["retrace"] == {"kernel": "scan_kernel<4,1,1,256,8,4,0>", "launches": 1, "dram_bytes_per_launch": 738400000}
    assert doc["kernels"]["gae"]["dram_bytes_per_launch"] == 1024
    assert bench.load_traffic(str(out))["gae"]["kernel"] == "scan_kernel<0,1,1,128,16,6,0>"
