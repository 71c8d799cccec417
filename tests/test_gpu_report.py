"""The error-aware speedup sweep on a GPU, cut down to one workload graph: every instance of the
ladder (ten shapes, three storage types) runs fused and unfused, agrees between the two at the
paper's strict level t = -5, and is scored."""
import pytest

from paper_2605_29357_b200 import report as R

pytestmark = pytest.mark.gpu


def test_sweep_of_one_graph_scores_every_instance():
    doc = R.run_sweep(device=0, steps=5, warmup=2, names=["c1"])
    assert doc["instances"] == 30 and doc["errors"] == []
    assert doc["correct_at_t-5"] == 30                     # fused and unfused agree at the strict level
    assert len(doc["rows"]) == 30 and all(r["kernels_unfused"] >= 4 for r in doc["rows"])
    assert set(doc["ES_t"]) == {str(t) for t in range(-10, 5)}
    assert doc["ES_t"]["-5"] == pytest.approx(doc["gmean_speedup_of_correct"])
    assert doc["AS"] > 0
