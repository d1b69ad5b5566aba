"""GPU: every configuration driver in its quick form, and the allocation parity on the numbers it measured:
the measured maximum prefill throughput and TPOT curve each driver stored beside its allocations are fed to the
oracle, which must reproduce every integer bit for bit and every double exactly (alloc_check.check_result)."""
import json

import pytest

from alloc_check import check_result

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["tiny", "8b", "long_input", "decode_heavy", "70b"])
def test_driver_allocations_match_the_oracle_on_measured_numbers(pdlib, name):
    import paper_2603_04716_b200.configs as cfgs
    res = json.loads(json.dumps(cfgs.RUNNERS[name](True)))       # as a result file would hold it
    n = check_result(res, pdlib)
    assert n >= {"tiny": 1, "8b": 1, "long_input": 1, "decode_heavy": 5, "70b": 2}[name]
    if name == "decode_heavy":
        # TPOT grows with the batch, so a tighter SLO never admits a larger batch
        per = res["allocation_per_tpot_slo_ms"]
        best = [(per[s].get("refined") or per[s])["feasible_batch"] for s in ("20", "35", "50", "75", "100") if per[s]["status"] == 0]
        assert best == sorted(best)
    if name == "long_input":
        assert all(abs(c["interpolated_s"] / c["measured_s"] - 1.0) < 0.25 for c in res["interpolation_check"])  # quick: 4-point grid


def test_chunked_prefill_sweep_inside_the_harness(pdlib):
    import paper_2603_04716_b200.configs as cfgs
    res = cfgs.run_chunked(True)
    sw = res["chunk_sweep"]
    assert sw["1024"]["chunks"] == 4 and sw["4096"]["chunks"] == 1
    # a larger chunk does not lower the maximum prefill throughput (beyond timing noise)
    assert sw["4096"]["prefill_max_tok_s"] > 0.95 * sw["1024"]["prefill_max_tok_s"]
