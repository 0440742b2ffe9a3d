"""Host logic of the stage timer: intervals rebuilt from the ordering events, union of
overlapping launches.  CPU only: events are stand-ins that carry a timestamp."""
from paper_2609_34555_b200.runner import StageTimer


class FakeEvent:
    def __init__(self, t_ms: float):
        self.t = t_ms

    def elapsed_time(self, other: "FakeEvent") -> float:
        return other.t - self.t


def test_busy_time_is_the_union_of_overlapping_launches():
    tm = StageTimer(stages=("recall",))
    base = FakeEvent(0.0)
    for a, b in ((1.0, 3.0), (2.0, 4.0), (6.0, 7.0), (6.5, 6.8)):
        tm.add("recall", FakeEvent(a), FakeEvent(b))
    assert abs(tm.busy_ms("recall", base) - (3.0 + 1.0)) < 1e-12
    s = tm.summary()["recall"]
    assert s["launches"] == 4 and abs(s["total_ms"] - (2 + 2 + 1 + 0.3)) < 1e-9


def test_light_summary_rebuilds_stage_intervals_from_ordering_events():
    """Two layers, two recall streams, two steps.  Times (ms) of the events diff done / recall
    landed / attention done per (step, layer) are chosen by hand; the expected intervals follow
    the rule: a stage starts when its stream is free and its input event has fired."""
    tm = StageTimer(light=True)
    base = FakeEvent(0.0)
    rec = [
        # layer, recall stream, diff done, recall landed, attention done
        (0, 0, 1.0, 5.0, 6.0),
        (1, 1, 2.0, 8.0, 9.0),
        (0, 0, 7.0, 12.0, 13.0),     # its recall can start at max(diff 7.0, stream-0 free 5.0) = 7.0
        (1, 1, 9.5, 14.0, 15.0),     # starts at max(diff 9.5, stream-1 free 8.0) = 9.5
    ]
    for layer, rs, td, tr, ta in rec:
        tm.records.append((layer, rs, FakeEvent(td), FakeEvent(tr), FakeEvent(ta)))
    out = tm.light_summary(base)
    # recall: first launch of each stream left out; (7,12) and (9.5,14): union 7..14
    assert out["recall"]["launches"] == 2
    assert abs(out["recall"]["total_ms"] - (5.0 + 4.5)) < 1e-9
    assert abs(out["recall"]["busy_ms"] - 7.0) < 1e-9
    # attention: starts at max(recall landed, previous attention done): (8,9), (12,13), (14,15)
    assert out["attn"]["launches"] == 3 and abs(out["attn"]["total_ms"] - 3.0) < 1e-9
    # select+diff: starts at max(previous diff done, this layer's previous attention done):
    # (1,2), (max(2, 6)=6, 7), (max(7, 9)=9, 9.5)
    sd = out["select_diff"]
    assert sd["launches"] == 3
    assert abs(sd["total_ms"] - (1.0 + 1.0 + 0.5)) < 1e-9
