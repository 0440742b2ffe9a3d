"""The interruptible layer-wise scheduler on a simulated GPU (no device needed): overlap depth
follows the recall time, and the three completion-detection modes order as the paper says
(Sec. 4.2.2): synchronous detection leaves the GPU idle between layers, asynchronous detection
resumes the offload batch late, semi-synchronous detection does neither."""
import math
import statistics

import pytest

from paper_2609_34555_b200.irq import MODES, simulate


@pytest.mark.parametrize("t_io", [100.0, 400.0, 1000.0])
def test_overlap_depth_follows_recall_time(t_io):
    rep, _ = simulate("semi", offload_layers=40, t_io=t_io, t_attn=40.0, t_ffn=80.0)
    t_layer = 120.0
    m = statistics.fmean(rep.depths[1:])
    assert abs(m - max(1, math.ceil(t_io / t_layer))) <= 1.0           # m = ceil(t_io / t_layer), give or take the phase
    assert rep.offload_layers == 40 and rep.normal_layers == sum(rep.depths)


def test_depth_adapts_to_a_varying_recall_load():
    loads = lambda layer: 150.0 if layer % 2 == 0 else 900.0            # light and heavy layers alternate
    rep, _ = simulate("semi", offload_layers=40, t_io=loads)
    even, odd = rep.depths[2::2], rep.depths[3::2]
    assert statistics.fmean(odd) > 2 * statistics.fmean(even)


def test_three_detection_modes_order_as_described():
    res = {m: simulate(m, offload_layers=60, t_io=400.0, launch_us=6.0) for m in MODES}
    idle = {m: res[m][1] for m in MODES}
    delay = {m: statistics.fmean(res[m][0].resume_delay_us) for m in MODES}
    # synchronous: the queue drains at every layer boundary -> the GPU idles most
    assert idle["sync"] > 2 * idle["semi"] and idle["sync"] > 2 * idle["async"]
    # asynchronous: layers already queued delay the switch back to the offload batch
    assert delay["async"] > 1.5 * delay["semi"]
    # semi-synchronous: bounded delay (less than one normal layer + launch) and little idling
    assert delay["semi"] < 120.0 + 3 * 6.0
    for m in MODES:
        assert res[m][0].offload_layers == 60
