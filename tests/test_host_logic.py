"""Host logic that needs no GPU: the bytes-per-element model of the roofline
against the traffic the paper prints, the rank partition, the workload shapes."""
import os

import pytest

import bench
from paper_2601_07876_b200 import sharding, workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden", "traffic_section_5_5.txt")


def _gold():
    vals = {}
    for line in open(GOLD):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            vals[k] = int(v)
    return vals


def test_bytes_model_matches_the_papers_traffic():
    g = _gold()
    per = bench.algorithmic_bytes_per_elem(4, 0, "last", 3)     # no lookahead
    assert per == 28 and per * g["p"] == g["total_bytes"]
    assert 16 * g["p"] == g["read_bytes"] and 12 * g["p"] == g["write_bytes"]


def test_bytes_model_lookahead_schedule():
    f = bench.algorithmic_bytes_per_elem
    # LAST, k=5: slow written at t=1, read+written on syncs, untouched otherwise
    assert [f(4, 5, "last", t) for t in range(1, 11)] == [32, 28, 28, 28, 36, 28, 28, 28, 28, 36]
    assert sum(f(4, 5, "last", t) for t in range(6, 11)) / 5 == 28 + 8 / 5
    # bf16 gradients: 2 bytes less
    assert f(2, 6, "last", 7) == 26 and f(2, 6, "last", 12) == 34
    # TRAJ_MEAN, k=4: first of window writes the sum, middle reads+writes, sync reads sum+slow, writes slow
    assert [f(4, 4, "traj_mean", t) for t in range(5, 9)] == [32, 36, 36, 40]
    assert f(4, 4, "traj_mean", 1) == 36
    # k = 1: both modes are the LAST rule on every step
    assert f(4, 1, "traj_mean", 1) == f(4, 1, "last", 1) == 36
    assert f(4, 1, "traj_mean", 2) == f(4, 1, "last", 2) == 36


def test_workload_shapes():
    want = {0: (1, 1_048_576), 1: (161, 25_557_032), 2: (32, 138_357_544),
            3: (152, 86_567_656), 4: (1000, 1_000_000_000)}
    for i, (n, total) in want.items():
        wl = W.get_workload(i)
        assert (len(wl.numel), wl.total) == (n, total)
    assert sum(1 for x in W.get_workload(1).numel if x < 1024) == 85
    assert max(W.get_workload(2).numel) == 102_760_448
    wl = W.get_workload(4)
    assert min(wl.numel) >= 1024 and max(wl.numel) <= 16 * 2 ** 20
    assert any(x % 4 for x in wl.numel)
    offs, total = W.element_offsets(wl)
    assert sum(1 for o in offs if o % 4) == 333            # every third tensor misaligned
    assert all(offs[i] + wl.numel[i] <= offs[i + 1] for i in range(len(offs) - 1))
    assert W.get_workload(4).numel == wl.numel             # seeded: same sizes every time


@pytest.mark.parametrize("world", [1, 2, 3, 8])
def test_partition_covers_every_element_once(world):
    numel = [5, 64, 1000, 3, 70001, 128]
    parts = sharding.partition_flat(numel, world, align=64)
    assert len(parts) == world
    seen = [[0] * n for n in numel]
    sizes = []
    for slices in parts:
        sizes.append(sum(b - a for _, a, b in slices))
        for t, a, b in slices:
            assert 0 <= a < b <= numel[t]
            for i in range(a, b):
                seen[t][i] += 1
    assert all(all(x == 1 for x in s) for s in seen)
    assert max(sizes) - min(sizes) <= 64 + 63
    flat = [(t, a) for slices in parts for t, a, _ in slices]
    assert flat == sorted(flat)                            # contiguous, in order


def _paper_constants():
    path = os.path.join(os.path.dirname(__file__), "golden", "constants_sections_4_and_5.txt")
    out = {}
    for line in open(path):
        line = line.split("#")[0].split()
        if len(line) == 2:
            out[line[0]] = float(line[1])
    return out


def test_library_defaults_and_oracle_follow_the_constants_the_paper_prints():
    import numpy as np
    from oracle import novak_oracle as O
    from paper_2601_07876_b200 import binding as B
    c = _paper_constants()
    h = B.Handle(beta1=c["beta1_default"], beta2=c["beta2_default"], eps=c["eps_default"])
    assert h.get_option(B.NOVAK_OPT_BETA1_TAU) == c["tau1"]
    assert h.get_option(B.NOVAK_OPT_BETA2_TAU) == c["tau2"]
    assert h.get_option(B.NOVAK_OPT_AUTO_LR_GAMMA) == c["auto_lr_gamma"]
    assert h.get_option(B.NOVAK_OPT_CLIP_THRESHOLD) == 0.0        # off unless asked for
    # Eq. 6 and the threshold of Eq. 8, in the library's plan and in the oracle
    o = O.Oracle(O.Config(beta1=c["beta1_default"], beta2=c["beta2_default"]), [np.zeros(1)])
    assert abs(h.plan(1).rho_inf - c["rho_inf_beta2_0.999"]) < 1e-9
    assert abs(o.scalars(1).rho_inf - c["rho_inf_beta2_0.999"]) < 1e-9
    for t in range(1, 40):
        for plan in (h.plan(t), o.scalars(t)):
            assert plan.rect_branch == (1 if plan.rho_t >= c["rectification_threshold"] else 0)
    assert [h.plan(t).rect_branch for t in (5, 6)] == [0, 1]
    # the clip ranges of Eq. 19 and Eq. 22, in the oracle
    for scale, lo_hi in ((1e-6, "low"), (1e6, "high")):
        o = O.Oracle(O.Config(lookahead_k=0, layer_adaptation=True, auto_lr=True),
                     [np.full(8, scale)])
        o.step([np.full(8, 1.0 / scale)])
        assert o.trust[0][0] == c[f"trust_clip_{lo_hi}"]
        # the gradient scale runs the other way: tiny parameters, huge gradient -> upper bound
        assert o.auto_scales[0] == c["auto_lr_clip_high" if lo_hi == "low" else "auto_lr_clip_low"]
    assert O.Config().tau1 == c["tau1"] and O.Config().tau2 == c["tau2"]
    assert O.Config().auto_lr_gamma == c["auto_lr_gamma"]
