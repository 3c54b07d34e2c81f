"""Host-side logic of bench.py that needs no GPU: which steps a run times, the config block both
arms print, the byte model, and the oracle baseline on every core (on a tiny workload)."""
import importlib.util
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench():
    spec = importlib.util.spec_from_file_location("_bench", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


class _Args:
    algorithm, grad_dtype = "alg1", "f32"


def test_step_window_holds_every_kind_of_step():
    bench = _bench()
    from paper_2202_06009_b200 import synth
    for name, make in synth.WORKLOADS.items():
        wl = make()
        steps = bench.step_window(wl, 20)
        assert len(steps) == 20 and steps == list(range(steps[0], steps[0] + 20))
        kinds = {(wl.in_T_u(t), wl.in_T_v(t)) for t in steps}
        assert (True, False) in kinds and (False, False) in kinds and (True, True) in kinds, name
        assert bench.step_window(wl, wl.steps) == list(range(wl.steps))          # a whole schedule starts at 0
    wl = synth.bert_large()
    assert bench.step_window(wl, 20)[0] == 61                                    # first local step of the schedule is t = 65


def test_both_arms_print_the_same_config_block():
    bench = _bench()
    from paper_2202_06009_b200 import synth
    wl = synth.bert_large()
    steps = bench.step_window(wl, 20)
    a, b = bench.config_block(wl, _Args, steps, 1), bench.config_block(wl, _Args, steps, 1)
    assert a == b and a["workload"] == "bert_large" and a["n_params"] == 336226108 and a["W"] == 16 and a["chunk"] == 4096
    assert "t=61..80" in a["schedule"] and "8 local" in a["schedule"] and "11 sync" in a["schedule"]


def test_byte_model():
    """The algorithmic bytes of the survey's table: 28 + 4/W per parameter and worker for a local
    step, 32 1/8 + 20 1/8 / W (+ a magnitude per chunk) for a fused sync step."""
    bench = _bench()
    n, W, chunk = 1 << 20, 16, 4096
    assert bench.local_step_bytes(n, W) == n * W * 28 + 4 * n
    per = bench.sync_step_bytes(n, W, chunk) / (n * W)
    assert abs(per - (32.125 + 20.125 / W + 4 / chunk + 4 / chunk / W)) < 1e-9
    assert abs(bench.sync_step_bytes(336226108, 16, 4096) / 1e9 - 179.59) < 0.01          # the 179.6 GB of a BERT-Large sync step
    assert bench.two_call_sync_bytes(n, W, chunk) > 1.5 * bench.sync_step_bytes(n, W, chunk)


def test_oracle_baseline_uses_the_cores_and_the_given_gradients():
    bench = _bench()
    import numpy as np
    import torch
    from paper_2202_06009_b200 import synth
    wl = synth.tiny(n=64 * 2048, W=2, chunk=2048, steps=8)
    stream = synth.GradientStream(wl, "cpu")
    asked = []

    def grads_of(t):
        asked.append(t)
        return stream.fill(t)

    value, cores, desc, s_per_step = bench.time_oracle(wl, [3, 4, 5], grads_of, synth.initial_params(wl, "cpu"), 1 << 25)
    assert asked == [3, 4, 5]
    assert cores == min(len(os.sched_getaffinity(0)), 64) and value > 0 and s_per_step > 0
    assert f"{cores} chunk ranges" in desc and "t=3..5" in desc


def test_traffic_ratios_are_the_ones_in_the_committed_profiles():
    """bench.py's roofline.traffic is a measured ratio times the algorithmic bytes: every ratio must be
    printed in the ncu summary it names, so that a re-captured kernel cannot leave a stale constant."""
    import os
    import bench
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    for kernel, (ratio, summary) in bench.DRAM_TRAFFIC_RATIO.items():
        path = os.path.join(root, "profiles", summary)
        assert os.path.exists(path), (kernel, summary)
        text = open(path).read()
        assert f"{ratio}" in text, (kernel, ratio, summary)
