"""The closed forms of the cost model against what the paper prints and proves (no GPU).

Printed values: Table 1's GPU specifications give the hardware ratios eta = 1.42 (H100 with
L40S) and 1.93 (H100 with A100) and the bounds 1.10x and 1.19x of Theorem 2 (Section 7.4).
Proved properties: Theorem 1 (no gain while b_bar >= b*, strictly increasing and bounded by
M / (M - M_weights) beyond), Theorem 2 (gain >= 1, = 1 under dominance, peak at the crossing
x*, bounded by (1 + sqrt(eta)) / 2, and the bound is approached for the worst price ratio).
"""
import math
import os

import numpy as np
import pytest

from paper_2609_14237_b200 import costmodel as cm

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_table1_eta.txt")


def load_golden():
    gpus, pairs = {}, []
    for line in open(GOLDEN):
        f = line.split("#")[0].split()
        if len(f) == 5:
            gpus[f[0]] = cm.gpu_from_table(f[0], *(float(x) for x in f[1:]))
        elif len(f) == 4:
            pairs.append((f[0], f[1], float(f[2]), float(f[3])))
    return gpus, pairs


def test_printed_hardware_ratios_and_bounds():
    gpus, pairs = load_golden()
    assert len(gpus) == 3 and len(pairs) == 2
    for a, b, eta, bound in pairs:
        assert round(cm.hardware_ratio(gpus[a], gpus[b]), 2) == eta
        assert cm.hardware_ratio(gpus[a], gpus[b]) == cm.hardware_ratio(gpus[b], gpus[a])
        assert round(cm.gain_het_bound(gpus[a], gpus[b]), 2) == bound


def test_roofline_and_attention_latency():
    assert cm.operator_latency(8e9, 1e12, 4e12, 1e15) == 2e-3          # memory-bound
    assert cm.operator_latency(8e6, 1e13, 4e12, 1e15) == 1e-2          # compute-bound
    m = cm.kv_bytes_per_request(32768, 1, 8, 128)
    assert m == 32768 * 4096
    assert cm.kv_bytes_per_request(32768, 1, 8, 128, window=4096) == 4096 * 4096
    assert cm.kv_bytes_per_request(100, 1, 8, 128, window=4096) == 100 * 4096
    assert math.isclose(cm.attention_latency(16, m, 6.5e12), 16 * m / 6.5e12)


def model():
    g = cm.gpu_from_table("H100", 3350, 80, 989, 3.49)
    p_act = 22e9 / 8            # activated parameters per request after 8-way sharding
    m_w = 235e9 * 2 / 8         # resident weights per GPU
    return g, p_act, m_w


def test_eq1_to_eq4_and_threshold_by_hand():
    g, p_act, m_w = model()
    m_kv = 2e9
    assert math.isclose(cm.cpt_hom(g, m_kv, p_act), g.cost / g.beta * m_kv + 2 * g.cost / g.flops * p_act)
    l40 = cm.gpu_from_table("L40S", 864, 48, 362.05, 1.09)
    assert math.isclose(cm.cpt_het(l40, g, m_kv, p_act), l40.alpha * m_kv + 2 * g.gamma * p_act)
    b_bar, b_max = cm.batch_limit(g, m_w, m_kv)
    assert math.isclose(b_bar, (80e9 - m_w) / 2e9) and b_max == math.floor(b_bar)
    want = g.alpha * m_kv + max(g.alpha * m_w / b_bar, 2 * g.gamma * p_act)
    assert math.isclose(cm.cpt_coloc(g, m_kv, p_act, m_w), want)
    assert math.isclose(cm.gemm_threshold(g, m_w, p_act), m_w * g.flops / (2 * p_act * g.beta))
    assert cm.cpt_coloc(g, 1.0, p_act, 90e9) == math.inf              # weights alone do not fit


def test_theorem1_no_gain_then_increasing_and_bounded():
    g, p_act, m_w = model()
    b_star = cm.gemm_threshold(g, m_w, p_act)
    bound = cm.gain_hom_bound(g, m_w)
    assert math.isclose(bound, 80e9 / (80e9 - m_w))
    free = g.mem - m_w
    xs = np.geomspace(free / (4 * b_star), free, 400)                 # m_kv from b_bar = 4 b* down to b_bar = 1
    gains = np.array([cm.gain_hom(g, x, p_act, m_w) for x in xs])
    b_bars = free / xs
    short = b_bars >= b_star
    assert short.any() and (~short).any()
    np.testing.assert_allclose(gains[short], 1.0, rtol=1e-12)          # part 1
    longer = gains[~short]
    assert (longer > 1.0).all() and (np.diff(longer) > 0).all()         # part 2
    assert (gains < bound).all() and gains[-1] > 0.5 * (1 + bound)      # part 3, and it gets close


def two_types(price_ratio=1.0):
    a = cm.Gpu("bw", 1.0, 4.0, 1.0, 1.0)                              # bandwidth-rich
    b = cm.Gpu("fl", price_ratio, 1.0, 1.0, 3.0)                      # compute-rich
    return a, b


def test_theorem2_gain_at_least_one_peaks_at_the_crossing_and_is_bounded():
    a, b = two_types(1.3)
    p_act = 0.5
    eta = cm.hardware_ratio(a, b)
    assert math.isclose(eta, 12.0)
    bound = cm.gain_het_bound(a, b)
    x_star = cm.het_crossing(a, b, p_act)
    assert math.isclose(cm.cpt_hom(a, x_star, p_act), cm.cpt_hom(b, x_star, p_act))
    xs = np.geomspace(x_star / 100, x_star * 100, 2001)
    gains = np.array([cm.gain_het([a, b], x, p_act) for x in xs])
    assert (gains >= 1.0 - 1e-12).all() and (gains <= bound + 1e-12).all()
    peak = int(np.argmax(gains))
    assert abs(math.log(xs[peak] / x_star)) < 0.01
    assert (np.diff(gains[:peak]) > 0).all() and (np.diff(gains[peak + 1:]) < 0).all()


def test_theorem2_no_gain_under_dominance():
    a = cm.Gpu("big", 1.0, 4.0, 1.0, 4.0)
    b = cm.Gpu("small", 1.0, 2.0, 1.0, 3.0)                           # worse on both metrics at equal price
    assert cm.het_crossing(a, b, 1.0) == math.inf
    for x in (0.01, 1.0, 100.0):
        assert math.isclose(cm.gain_het([a, b], x, 1.0), 1.0)


def test_theorem2_bound_is_attained_for_the_worst_price_ratio():
    """sup over prices and sequence lengths of G_het equals (1 + sqrt(eta)) / 2."""
    best = 0.0
    for r in np.geomspace(0.05, 20, 400):
        a, b = two_types(r)
        x_star = cm.het_crossing(a, b, 1.0)
        if math.isfinite(x_star) and x_star > 0:
            best = max(best, cm.gain_het([a, b], x_star, 1.0))
    bound = cm.gain_het_bound(*two_types())
    assert best <= bound + 1e-12 and best > bound * (1 - 1e-3)


def test_cad_feasibility_condition():
    h100 = cm.gpu_from_table("H100", 3350, 80, 989, 3.49)
    assert math.isclose(cm.cad_attn_latency_max(h100, 4), 80e9 / (4 * 3350e9))
    assert math.isclose(cm.cad_rest_latency_min(h100, 30e9), 30e9 / 3350e9)
    assert cm.cad_feasible(h100, 2, h100, 30e9)                        # 11.9 ms >= 9.0 ms
    assert not cm.cad_feasible(h100, 4, h100, 30e9)                    # 6.0 ms < 9.0 ms
    faster_rest = cm.with_measured_bandwidth(h100, 8e12)
    assert cm.cad_feasible(h100, 4, faster_rest, 30e9)                 # more bandwidth on the GEMM side helps


def test_affine_latency_fit_recovers_floor_and_bandwidth():
    """T = t0 + D / beta through exact points gives t0 and beta back; noise moves them little; bad inputs raise."""
    t0, beta = 15e-6, 7.1e12
    sizes = [4e6, 68e6, 270e6, 1.07e9, 4.3e9, 17e9]
    exact = [(d, t0 + d / beta) for d in sizes]
    f0, fb = cm.fit_affine_latency(exact)
    assert abs(f0 - t0) < 1e-12 and abs(fb / beta - 1) < 1e-9
    noisy = [(d, t * (1 + 0.01 * (-1) ** i)) for i, (d, t) in enumerate(exact)]
    n0, nb = cm.fit_affine_latency(noisy)
    assert abs(nb / beta - 1) < 0.03 and abs(n0 - t0) < 10e-6
    assert cm.attention_latency_affine(64, 2560 * 4096, t0, beta) == pytest.approx(t0 + 64 * 2560 * 4096 / beta)
    assert cm.attention_latency_affine(64, 2560 * 4096, 0.0, beta) == pytest.approx(cm.attention_latency(64, 2560 * 4096, beta))
    for bad in ([(1e6, 1e-5)], [(1e6, 1e-5), (1e6, 2e-5)], [(1e6, 2e-5), (2e6, 1e-5)]):
        with pytest.raises(ValueError):
            cm.fit_affine_latency(bad)
