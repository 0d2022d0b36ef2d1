"""The utilisation report's arithmetic on hand-made event lists (no GPU)."""
import numpy as np

from paper_2609_21483_b200 import timeline as tl


def _rec(t0, t1, kind, ident=0, extra=0, base=0):
    return [(base + t0) & 0xFFFFFFFF, (base + t1) & 0xFFFFFFFF, (kind << 24) | ident, extra]


def _trace(base=0):
    ctas = [[], [], [], []]
    for c in range(4):
        ctas[c].append(_rec(0, 100, tl.EV_ROUTE, base=base))
        ctas[c].append(_rec(100, 200, tl.EV_SETUP, base=base))
    ctas[0].append(_rec(200, 1200, tl.EV_MMA, base=base))           # pair (0, 1) runs one GEMM main loop
    ctas[2].append(_rec(200, 700, tl.EV_DISPATCH, base=base))
    ctas[2].append(_rec(700, 1200, tl.EV_WAIT_CHUNK, base=base))    # waiting is idle time
    ctas[3].append(_rec(1200, 1700, tl.EV_COMBINE, base=base))
    return [np.array(c, dtype=np.uint32) for c in ctas]


def test_report_on_a_known_timeline():
    rep = tl.analyse(_trace())
    assert rep["window_us"] == 1.6 and rep["routing_us"] == 0.1
    assert abs(rep["movement_active"] - 0.625) < 1e-12
    assert abs(rep["tensor_active"] - 0.625) < 1e-12
    assert abs(rep["overlap_ratio"] - 0.3125) < 1e-12
    assert abs(rep["sm_busy"] - 0.53125) < 1e-12
    assert abs(rep["sm_busy_min"] - 600 / 1600) < 1e-12
    assert abs(rep["mean_ctas_moving"] - 0.625) < 1e-12
    assert abs(rep["mean_ctas_gemm"] - 1.25) < 1e-12


def test_counter_wrap_does_not_change_the_report():
    a = tl.analyse(_trace())
    b = tl.analyse(_trace(base=(1 << 32) - 650))      # the 32-bit time stamps wrap in the middle of the kernel
    for k in ("window_us", "movement_active", "tensor_active", "overlap_ratio", "sm_busy"):
        assert abs(a[k] - b[k]) < 1e-12, k


def test_accumulator_wait_is_not_tensor_work():
    tr = _trace()
    tr[0][2, 3] = 300                                   # the main loop first waited 300 ns for an accumulator
    rep = tl.analyse(tr)
    assert abs(rep["tensor_active"] - 700 / 1600) < 1e-12
    assert abs(rep["overlap_ratio"] - 200 / 1600) < 1e-12


def test_rates_use_the_live_time_of_each_kind():
    rep = tl.analyse(_trace(), {"T": 8, "H": 128, "I": 64, "k": 2, "S": 0})
    P = 16
    assert abs(rep["dispatch_GBps"] - 2 * P * 128 * 2 / 0.5 / 1e3) < 1e-9
    assert abs(rep["combine_GBps"] - (P + 8) * 128 * 2 / 0.5 / 1e3) < 1e-9
    assert abs(rep["gemm_TFLOPs"] - P * 6 * 128 * 64 / 1.0 / 1e6) < 1e-9


def test_ascii_timeline_marks_the_roles():
    txt = tl.ascii_timeline(_trace(), width=17).splitlines()
    assert len(txt) == 5
    assert txt[1].split()[1].startswith("RsGGGGGGGGGG")      # CTA 0: routing, set-up, GEMM
    assert "D" in txt[3] and "C" not in txt[3]
    assert txt[4].rstrip().endswith("CCCCC")
