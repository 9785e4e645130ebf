"""Host-side entry points of the library (no device work, so they run without a GPU) against the oracle in
oracle/schedule.py and against the numbers the paper prints."""
import random

import numpy as np
import pytest

import paper_2003_10735_b200 as st
from oracle import schedule as sch
from test_schedule_pins import G, L, MIN, MAX, hand_traces


def lat():
    return st.st_latencies(L.t_si, L.t_sd, L.t_ti, L.t_net)


def test_next_stride_matches_the_oracle_everywhere():
    rnd = random.Random(0)
    for _ in range(3000):
        thr = rnd.choice([0.5, 0.8, 0.9, rnd.uniform(0.05, 0.95)])
        lo = rnd.randint(1, 16); hi = lo + rnd.randint(0, 100)
        s = rnd.randint(lo, hi); m = rnd.choice([0.0, 1.0, thr, rnd.random()])
        assert st.st_next_stride(s, m, thr, lo, hi) == sch.next_stride(s, m, thr, lo, hi), (s, m, thr, lo, hi)


@pytest.mark.parametrize("delay", [1, 3, 8, 40])
def test_client_schedule_matches_the_oracle(delay):
    rnd = random.Random(delay)
    metrics = [rnd.random() for _ in range(700)]
    for n in (0, 1, 7, 8, 9, 500, 5000):
        assert st.st_client_schedule(n, metrics, 0.8, MIN, MAX, delay) == sch.client_schedule(n, metrics, 0.8, MIN, MAX, delay)


def test_client_schedule_reproduces_the_hand_worked_sequences():
    for n, delay, metrics, keys in hand_traces():
        assert st.st_client_schedule(n, metrics, G["threshold"], MIN, MAX, delay) == keys, (n, delay, metrics)


def test_client_schedule_errors():
    with pytest.raises(st.StError) as ei:
        st.st_client_schedule(100, [0.5], 0.8, 8, 64, 1)                  # second key frame has no metric
    assert ei.value.status == st.ST_ERR_INVALID_ARG
    for bad in (dict(threshold=1.0), dict(min_stride=0), dict(max_stride=4), dict(delay=0)):
        kw = dict(threshold=0.8, min_stride=8, max_stride=64, delay=1); kw.update(bad)
        with pytest.raises(st.StError):
            st.st_client_schedule(10, [0.5] * 4, **kw)


def test_bounds_reproduce_the_papers_numbers_and_the_oracle():
    U = int(G["max_updates"])
    lo, hi = st.st_throughput_bounds(lat(), MIN, MAX, U)
    assert round(hi, 2) == G["fps_upper"] and lo > G["fps_floor"]
    assert (lo, hi) == pytest.approx(sch.throughput_bounds(L, MIN, MAX, U), rel=1e-14)
    mb = G["s_net_bytes"] * 8 / 1e6
    tlo, thi = st.st_traffic_bounds(lat(), mb, MIN, MAX, U)
    assert round(tlo, 2) == G["mbps_lower"] and round(thi, 1) == G["mbps_upper"]
    assert (tlo, thi) == pytest.approx(sch.traffic_bounds(L, mb, MIN, MAX, U), rel=1e-14)
    assert st.st_choose_max_updates(lat(), MIN, MAX, G["fps_floor"]) == U
    for floor in (1.0, 3.0, 5.5, 6.9, 50.0):
        assert st.st_choose_max_updates(lat(), MIN, MAX, floor) == sch.choose_max_updates(L, MIN, MAX, floor, limit=1 << 20)
    with pytest.raises(st.StError):
        st.st_throughput_bounds(st.st_latencies(0.0, 0.013, 0.044, 0.303), MIN, MAX, U)
    with pytest.raises(st.StError):
        st.st_traffic_bounds(lat(), 1.0, 64, 8, U)
