"""Host-only checks around bench.py and the sources that travel to multi-GPU runs."""
import json
import os
import re
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line_with_the_contract_keys():
    """`bench.py --impl reference` times the CPU oracle; here on a small sample so that it takes seconds."""
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "bert_base_fc",
                        "--reference-rows", "64", "--steps", "2", "--warmup", "1", "--reference-budget-s", "20"],
                       cwd=ROOT, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "q8_linear_int8_tops" and d["unit"] == "TOPS"
    assert d["value"] > 0 and d["higher_is_better"] is True and d["dtype"] == "int8" and d["data"] == "synthetic"
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["config"]["workload"] == "bert_base_fc" and 1 <= d["steps"] <= 2
    assert d["config"]["steps_requested"] == 2


def test_reference_arm_does_no_work_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_no_load_uses_cluster_multicast():
    """The same sources run as replicas on several GPUs, so no TMA or bulk load may use cluster multicast; the only
    multicast qualifier allowed in the tree is the one on tcgen05.commit (a barrier arrival in both CTAs of a pair)."""
    csrc = os.path.join(ROOT, "paper_1910_06188_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        text = open(os.path.join(csrc, name)).read()
        code = re.sub(r"//[^\n]*", "", text)
        for m in re.finditer(r"\"([^\"]*multicast::cluster[^\"]*)\"", code):
            assert "tcgen05.commit" in m.group(1), f"{name}: {m.group(1)}"
        assert not re.search(r"cp\.async\.bulk[^\"]*multicast", code), name


def test_bench_and_product_do_not_read_working_files():
    for path in ["bench.py", "__graft_entry__.py"] + [os.path.join("paper_1910_06188_b200", f)
                                                      for f in os.listdir(os.path.join(ROOT, "paper_1910_06188_b200")) if f.endswith(".py")]:
        text = open(os.path.join(ROOT, path)).read()
        assert not re.search(r"[\"'/]_work[/\"']", text), path   # the folder of working files, not e.g. new_workspace
