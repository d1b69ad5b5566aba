"""CPU: allocation parity on measured numbers.

tests/golden/measured/*.json are result files of the configuration drivers
(`python -m paper_2603_04716_b200.configs <name> --out FILE`): measured prefill throughputs and TPOT curves
of one B200 together with the allocations pd_allocate derived from them.  The measured numbers are inputs
to both sides; every expected value is computed here, by the oracle, from those inputs.  The library's
host code (no GPU needed) is run on the same inputs as well."""
import glob
import json
import os

import pytest

from alloc_check import check_result

HERE = os.path.dirname(os.path.abspath(__file__))
FILES = sorted(glob.glob(os.path.join(HERE, "golden", "measured", "*.json")))


@pytest.mark.parametrize("path", FILES, ids=[os.path.basename(f) for f in FILES])
def test_stored_measurements_reproduce_under_the_oracle(pdlib, path):
    with open(path) as f:
        res = json.load(f)
    assert check_result(res, pdlib) >= 1


def test_every_configuration_has_a_measurement_file():
    names = {os.path.basename(f).split(".")[0] for f in FILES}
    assert {"tiny", "8b", "long_input", "decode_heavy", "70b"} <= names
