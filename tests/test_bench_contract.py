"""The benchmark's reference arm (the oracle timed on the host cores) runs without a GPU: its JSON line is checked
here; the GPU arm's line is checked on a GPU machine."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(args, timeout=600):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, cwd=ROOT, capture_output=True,
                         text=True, timeout=timeout)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, out.stdout[-2000:]
    return json.loads(lines[0])


def test_reference_arm_line_on_cpu():
    d = _run(["--impl", "reference", "--workload", "C1", "--steps", "2", "--warmup", "1"])
    assert d["impl"] == "reference" and d["unit"] == "trees/s" and d["higher_is_better"] is True
    assert d["value"] > 0 and d["steps"] == 2 and d["warmup"] == 1 and d["n_gpus"] == 1
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert "workload" in d["config"]


@pytest.mark.gpu
def test_gpu_arm_line():
    d = _run(["--workload", "C2", "--steps", "40", "--warmup", "5", "--no-cpu-baseline"])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "gpu_launches", "roofline", "e2e", "clocks"):
        assert key in d, key
    assert d["steps"] == 40 and d["warmup"] == 5 and d["gpu_launches"] == 4 * 40 and d["vs_baseline"] is None
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert d["e2e"]["h2d_bytes_per_step"] > 0 and d["e2e"]["d2h_bytes_per_step"] > 0
    assert abs(d["value"] - 16 / (d["ms_per_step"] * 1e-3)) / d["value"] < 1e-6
    assert d["status_or"] == 0


def test_adversarial_rows_are_seeded_and_whole():
    """The rows of `bench.py --rows`: named, of the asked width at small and full widths, the same for the same seed."""
    import torch
    sys.path.insert(0, ROOT)
    import graft_inputs as gi
    for V in (4099, 40003):
        a = gi.adversarial_rows(V, torch.Generator().manual_seed(11))
        b = gi.adversarial_rows(V, torch.Generator().manual_seed(11))
        assert len(a) >= 40 and len({n for n, _ in a}) == len(a), [n for n, _ in a]
        for (na, ra), (nb_, rb) in zip(a, b):
            assert na == nb_ and ra.shape == (V,) and ra.dtype == torch.float32
            assert torch.equal(torch.nan_to_num(ra, neginf=-1e30), torch.nan_to_num(rb, neginf=-1e30))
            assert not torch.isnan(ra).any() and not torch.isposinf(ra).any()


@pytest.mark.gpu
def test_gpu_rows_line():
    d = _run(["--rows", "--workload", "C2", "--steps", "1"])
    assert d["shape"] == "C2" and len(d["times"]) >= 40
    assert all(t["vocab_pass_us"] > 0 and t["status_or"] == 0 for t in d["times"])
