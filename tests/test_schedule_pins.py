"""Pins for the oracle of the host-side pieces (Algorithm 2, Algorithm 4's control flow, Section 4.4's bounds):
the numbers the paper prints for its own configuration, the geometric description of Algorithm 2's two lines,
the general formula (Eq. 2) evaluated at the corner cases the bounds are derived from, and hand traces."""
import os

import pytest

from oracle import schedule as sch

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "section_5_3_bounds.txt")


def golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                k, v = line.split()
                out[k] = float(v)
    return out


G = golden()
L = sch.Latencies(G["t_si"], G["t_sd"], G["t_ti"], G["t_net"])
MIN, MAX = int(G["min_stride"]), int(G["max_stride"])


def test_paper_prints_6_99_fps_as_maximum_throughput():
    assert round(sch.throughput_bounds(L, MIN, MAX, 8)[1], 2) == G["fps_upper"]


def test_paper_picks_max_updates_8_for_a_5_fps_floor():
    assert sch.choose_max_updates(L, MIN, MAX, G["fps_floor"]) == int(G["max_updates"])
    lo8, lo9 = sch.throughput_bounds(L, MIN, MAX, 8)[0], sch.throughput_bounds(L, MIN, MAX, 9)[0]
    assert lo8 > 5.0 > lo9
    assert sch.throughput_bounds(L, MIN, MAX, 8)[1] - lo8 < 2.0          # "within 2 FPS"


def test_paper_prints_2_53_and_21_2_mbps_as_traffic_bounds():
    lo, hi = sch.traffic_bounds(L, G["s_net_bytes"] * 8 / 1e6, MIN, MAX, int(G["max_updates"]))   # megabits per key frame
    assert round(lo, 2) == G["mbps_lower"] and round(hi, 1) == G["mbps_upper"]


def test_bounds_are_the_general_formula_at_its_corner_cases():
    # Eq. 2 with the k, d, t_c of the four corner cases must reproduce the closed-form bounds
    n, U, s_net = 6400, 8, 3.0
    tc_lo, tc_hi = sch.t_c_bounds(L, MIN)
    t = sch.t_total(L, n, n / MIN, n / MIN * U, tc_hi, MIN)              # slowest: most keys, most steps, no concurrency
    assert n / t == pytest.approx(sch.throughput_bounds(L, MIN, MAX, U)[0], rel=1e-12)
    t = sch.t_total(L, n, n / MAX, 0, tc_lo, MIN)                         # fastest: fewest keys, no steps, full concurrency
    assert n / t == pytest.approx(sch.throughput_bounds(L, MIN, MAX, U)[1], rel=1e-12)
    t = sch.t_total(L, n, n / MAX, n / MAX * U, tc_hi, MIN)              # least traffic
    assert (n / MAX) * s_net / t == pytest.approx(sch.traffic_bounds(L, s_net, MIN, MAX, U)[0], rel=1e-12)
    t = sch.t_total(L, n, n / MIN, 0, tc_lo, MIN)                         # most traffic
    assert (n / MIN) * s_net / t == pytest.approx(sch.traffic_bounds(L, s_net, MIN, MAX, U)[1], rel=1e-12)
    assert tc_lo <= tc_hi


def test_next_stride_lines_pass_through_the_stated_points():
    T = G["threshold"]
    assert sch.next_stride_ratio(0.0, T) == 0.0                           # (0, 0)
    assert sch.next_stride_ratio(T, T) == pytest.approx(1.0)              # (THRESHOLD, 1) on the right-hand line
    assert sch.next_stride_ratio(T - 1e-12, T) == pytest.approx(1.0)      # ... and the left-hand line meets it
    assert sch.next_stride_ratio(1.0, T) == pytest.approx(2.0)            # (1, 2)
    assert sch.next_stride_ratio(0.4, T) == pytest.approx(0.5) and sch.next_stride_ratio(0.9, T) == pytest.approx(1.5)
    # monotone in the metric
    r = [sch.next_stride_ratio(i / 100, T) for i in range(101)]
    assert all(b >= a for a, b in zip(r, r[1:]))


def test_next_stride_clamps_and_truncates():
    T = G["threshold"]
    assert sch.next_stride(8, 0.0, T, MIN, MAX) == MIN                   # vanishing stride is held at MIN_STRIDE
    assert sch.next_stride(64, 1.0, T, MIN, MAX) == MAX                  # diverging stride is held at MAX_STRIDE
    assert sch.next_stride(16, 1.0, T, MIN, MAX) == 32 and sch.next_stride(16, 0.4, T, MIN, MAX) == 8
    assert sch.next_stride(10, 0.85, T, MIN, MAX) == 12                  # 1.25 * 10 = 12.5 -> 12 whole frames
    assert sch.next_stride(16, T, T, MIN, MAX) == 16                     # at the threshold the stride stays


def hand_traces():
    """(n_frames, delay, metrics, key frames) of every case in tests/golden/client_schedule_traces.txt."""
    out = []
    with open(os.path.join(os.path.dirname(GOLDEN), "client_schedule_traces.txt")) as f:
        for line in f:
            if not line.strip() or line.startswith("#"):
                continue
            head, metrics, keys = line.split("|")
            n, delay = (int(t) for t in head.split())
            out.append((n, delay, [float(t) for t in metrics.split()], [int(t) for t in keys.split()]))
    return out


def test_client_schedule_hand_traces():
    traces = hand_traces()
    assert len(traces) >= 9
    for n, delay, metrics, keys in traces:
        assert sch.client_schedule(n, metrics, G["threshold"], MIN, MAX, delay) == keys, (n, delay, metrics)


@pytest.mark.parametrize("delay", [1, 4, 8, 50])
def test_client_schedule_invariants(delay):
    import random
    rnd = random.Random(delay)
    metrics = [rnd.random() for _ in range(400)]
    keys = sch.client_schedule(3000, metrics, 0.8, 8, 64, delay)
    assert keys[0] == 0
    gaps = [b - a for a, b in zip(keys, keys[1:])]
    assert all(8 <= g <= 64 for g in gaps) and len(set(gaps)) > 3
