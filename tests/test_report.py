"""The error-aware speedup arithmetic (rectified speedup, ES_t, AS, the weights and the
tolerance ladder) against what the paper fixes: its printed weights and tolerances, the Eager
row of its main table, closed forms, and the factored form of its appendix.  CPU only."""
import math
import os
import random

import numpy as np
import pytest

from paper_2605_29357_b200 import report as R

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_weights_are_the_papers():
    assert R.t_values() == list(range(-10, 5))                      # t = -10 .. |E| + 1 with |E| = 3
    assert [R.weight(t) for t in (-10, -7, -6)] == [0.001] * 3      # extreme regime
    assert [R.weight(t) for t in (-5, -4, -3)] == [1.0] * 3         # strict-correctness regime
    for t in (-2, -1, 0, 1, 2, 3):
        assert R.weight(t) == pytest.approx(0.8 ** (t + 3))          # relaxed regime
    assert R.weight(4) == 0.001
    assert sum(R.weight(t) for t in R.t_values()) == pytest.approx(0.006 + 3 + 0.8 + 0.64 + 0.512 + 0.4096 + 0.32768 + 0.262144)


def test_tolerance_ladder_matches_the_printed_reference_points():
    rows = {r[0]: r for r in _gold("tolerance_ladder.txt")}
    for dtype, key in (("bf16", "bfloat16"), ("f16", "float16"), ("f32", "float32")):
        atol, rtol = R.tolerance(dtype, -5)
        assert atol == pytest.approx(float(rows[key][3]))
        assert float(f"{rtol:.1e}") == float(rows[key][2])            # the paper prints two digits
        assert R.tolerance(dtype, 0) == (1.0, 1.0)
        assert R.tolerance(dtype, 3) == (1.0, 1.0)                    # beyond 0 only categories are forgiven
        a10, r10 = R.tolerance(dtype, -10)
        assert a10 == pytest.approx(1e-10) and r10 == pytest.approx(rtol ** 2)   # log-linear in t
    assert R.tolerance("int", -5) == (0.0, 0.0)


def test_eager_row_scores_one():
    """Speedup 1 and correct everywhere: ES_t = 1 for every t and AS = 1.000 (main table, Eager)."""
    inst = [R.Instance(f"g{i}", 1.0, -10) for i in range(7)]
    assert all(R.es(inst, t) == pytest.approx(1.0) for t in R.t_values())
    assert R.aggregated_speedup(inst) == pytest.approx(1.0)


def test_rectified_speedup_cases():
    ok_fast = R.Instance("a", 2.5, -10)
    ok_slow = R.Instance("b", 0.5, -10)
    assert R.rectified_speedup(ok_fast, -5) == 2.5
    assert R.rectified_speedup(ok_slow, -5) == 0.5                              # p = 0: the slowdown itself
    assert R.rectified_speedup(ok_slow, -5, p=0.5) == pytest.approx(0.5 ** 1.5)
    loose = R.Instance("c", 3.0, -2)                    # passes the ladder only from t = -2 on
    assert R.rectified_speedup(loose, -3) == 0.1 and R.rectified_speedup(loose, -2) == 3.0
    assert R.rectified_speedup(loose, 2) == 3.0
    wrong = R.Instance("d", 3.0, None, error=1)         # fails even at t = 0: accuracy error
    assert R.rectified_speedup(wrong, 0) == 0.1 and R.rectified_speedup(wrong, 1) == 1.0
    nocompile = R.Instance("e", None, None, error=2)
    assert [R.rectified_speedup(nocompile, t) for t in (-5, 1, 2, 3)] == [0.1, 0.1, 1.0, 1.0]
    crash = R.Instance("f", None, None, error=3)
    assert [R.rectified_speedup(crash, t) for t in (2, 3, 4)] == [0.1, 1.0, 1.0]


def test_closed_form_with_a_fraction_of_errors():
    # 3 of 10 fail to compile (category 2), the rest run at speedup 1: ES_t = b^(0.3 [t < 2])
    inst = [R.Instance(f"ok{i}", 1.0, -10) for i in range(7)] + [R.Instance(f"x{i}", None, None, error=2) for i in range(3)]
    for t in R.t_values():
        assert R.es(inst, t) == pytest.approx(0.1 ** (0.3 if t < 2 else 0.0))
    wsum = sum(R.weight(t) for t in R.t_values())
    wlow = sum(R.weight(t) for t in R.t_values() if t < 2)
    assert R.aggregated_speedup(inst) == pytest.approx(0.1 ** (0.3 * wlow / wsum))
    assert R.fast_p(inst, 0.99) == pytest.approx(0.7)


def test_factored_form_of_the_appendix():
    """ES_t = alpha^(lambda (1 - eta)) beta^(lambda eta (p + 1)) gamma_t^(1 - lambda): geometric means of
    the correct-and-fast speedups, the correct-but-slow ones and the penalty factors."""
    rnd = random.Random(3)
    inst = []
    for i in range(40):
        kind = rnd.random()
        if kind < 0.5:
            inst.append(R.Instance(f"f{i}", 1.0 + rnd.random() * 3, -10))
        elif kind < 0.75:
            inst.append(R.Instance(f"s{i}", 0.2 + rnd.random() * 0.7, -10))
        else:
            inst.append(R.Instance(f"e{i}", None, None, error=rnd.choice([1, 2, 3])))
    b, p = 0.1, 0.25
    fast = [i.speedup for i in inst if i.error == 0 and i.speedup >= 1]
    slow = [i.speedup for i in inst if i.error == 0 and i.speedup < 1]
    errs = [i for i in inst if i.error]
    n = len(inst); lam = (len(fast) + len(slow)) / n; eta = len(slow) / (len(fast) + len(slow))
    gm = lambda v: math.exp(sum(math.log(x) for x in v) / len(v))
    for t in R.t_values():
        gamma = b ** (sum(1 for e in errs if t < e.error) / len(errs))
        want = gm(fast) ** (lam * (1 - eta)) * gm(slow) ** (lam * eta * (p + 1)) * gamma ** (1 - lam)
        assert R.es(inst, t, b, p) == pytest.approx(want, rel=1e-12)


def test_strictest_passing_level():
    ref = np.ones(8)
    assert R.strictest_passing_t(ref, ref, "f32") == -10
    # |err| = 3e-4 on a reference of 1: t = -3 allows 1e-3 + 10^(-3 * 5.886 / 5), t = -4 only 1.2e-4
    got = ref.copy(); got[3] += 3e-4
    assert R.strictest_passing_t(got, ref, "f32") == -3
    # bf16: rtol(t) = 10^(0.3592 t) is 5.8e-4 at t = -9 and 2.6e-4 at t = -10
    assert R.strictest_passing_t(got, ref, "bf16") == -9
    got[3] = 5.0
    assert R.strictest_passing_t(got, ref, "f32") is None           # 4 > atol(0) + rtol(0) * 1 = 2
    assert R.strictest_passing_t(np.array([1, 2]), np.array([1, 2]), "int") == -10
    assert R.strictest_passing_t(np.array([1, 3]), np.array([1, 2]), "int") is None
    assert R.strictest_passing_t(np.array([np.nan, np.inf]), np.array([np.nan, np.inf]), "f32") == -10
    assert R.strictest_passing_t(np.array([0.0, np.inf]), np.array([np.nan, np.inf]), "f32") is None


def test_summary_document():
    inst = [R.Instance("a", 4.0, -10), R.Instance("b", 1.0, -10), R.Instance("c", 9.0, -4)]
    doc = R.summarise(inst)
    assert doc["instances"] == 3 and doc["correct_at_t-5"] == 2
    assert doc["gmean_speedup_of_correct"] == pytest.approx(2.0)
    assert doc["ES_t"]["-5"] == pytest.approx((4.0 * 1.0 * 0.1) ** (1 / 3))
    assert doc["ES_t"]["-4"] == pytest.approx((4.0 * 1.0 * 9.0) ** (1 / 3))
    assert set(doc["ES_t"]) == {str(t) for t in range(-10, 5)}
