"""The promotion rule of the evaluation-spec harness (verified / admissible / promoted), on CPU."""
from paper_2609_35140_b200 import audit


def _spec():
    base = {k: 1.0 for k in audit.workload_names()}
    T = audit.aggregate(base)
    return {"baseline_ms": base, "baseline_T_ms": T, "incumbent_T_ms": T, "max_slowdown": 1.1,
            "hashes": {"c1": {"a": "h1", "b": "h2"}}}


def test_grid_is_the_papers_per_operator_grid():
    names = audit.workload_names()
    assert len(names) == 4 + 16 and len(set(names)) == 20
    assert "prefill_16384_bs1" in names and "decode_ctx8192_bs16" in names and "decode_ctx128_bs1" in names
    assert audit.aggregate({"a": 1.5, "b": 2.0}) == 3.5
    assert audit.aggregate({"a": 1.5, "b": 2.0}, {"a": 2.0}) == 5.0


def test_faster_everywhere_is_promoted():
    spec = _spec()
    lat = {k: 0.9 for k in spec["baseline_ms"]}
    v = audit.judge(spec, lat, True, "c1", {"a": "h1", "b": "h2"})
    assert v["verified"] and v["admissible"] and v["promoted"] and v["bitwise_preserved"] is True
    assert abs(v["speedup_over_baseline"] - 1 / 0.9) < 1e-12


def test_one_workload_over_the_limit_is_not_admissible_even_if_the_sum_improves():
    spec = _spec()
    lat = {k: 0.5 for k in spec["baseline_ms"]}
    lat["decode_ctx128_bs1"] = 1.2
    v = audit.judge(spec, lat, True, "c1", {"a": "h1", "b": "h2"})
    assert v["verified"] and not v["admissible"] and not v["promoted"]
    assert list(v["over_limit"]) == ["decode_ctx128_bs1"]


def test_within_limits_but_not_faster_is_admissible_not_promoted():
    spec = _spec()
    lat = {k: 1.05 for k in spec["baseline_ms"]}
    v = audit.judge(spec, lat, True, "c1", {"a": "h1", "b": "h2"})
    assert v["admissible"] and not v["promoted"]
    tie = audit.judge(spec, dict(spec["baseline_ms"]), True, "c1", {"a": "h1", "b": "h2"})
    assert tie["admissible"] and not tie["promoted"]            # ties do not replace the incumbent


def test_the_gate_has_no_absolute_slack():
    spec = _spec()
    lat = dict(spec["baseline_ms"])
    lat["decode_ctx128_bs1"] = 1.1                      # exactly at the limit: still admissible
    assert audit.judge(spec, lat, True, "c1", {"a": "h1", "b": "h2"})["admissible"]
    lat["decode_ctx128_bs1"] = 1.1005                   # 0.5 us over on a 1 ms workload: not admissible
    v = audit.judge(spec, lat, True, "c1", {"a": "h1", "b": "h2"})
    assert not v["admissible"] and list(v["over_limit"]) == ["decode_ctx128_bs1"]


def test_failed_checks_or_changed_bits_are_not_verified():
    spec = _spec()
    lat = {k: 0.5 for k in spec["baseline_ms"]}
    assert not audit.judge(spec, lat, False, "c1", {"a": "h1", "b": "h2"})["verified"]
    changed = audit.judge(spec, lat, True, "c1", {"a": "h1", "b": "XX"})
    assert changed["bitwise_preserved"] is False and not changed["verified"] and not changed["promoted"]
    # another contract id has no recorded hashes: preservation is undetermined, not a failure
    other = audit.judge(spec, lat, True, "c2", {"a": "zz"})
    assert other["bitwise_preserved"] is None and other["verified"] and other["promoted"]


def test_incomplete_measurements_are_not_admissible():
    spec = _spec()
    lat = {k: 0.5 for k in spec["baseline_ms"]}
    del lat["prefill_1024_bs1"]
    v = audit.judge(spec, lat, True, "c1", {"a": "h1", "b": "h2"})
    assert v["verified"] and not v["admissible"] and v["missing"] == ["prefill_1024_bs1"]


import json
import os

import pytest


@pytest.mark.gpu
def test_recorded_hashes_are_preserved_and_entry_points_agree():
    """Bitwise preservation: the outputs on the fixed seeded inputs hash to what was recorded for
    this contract id (a schedule-only change must not move them), and prefill / decode rows equal
    the packed forward's rows."""
    from paper_2609_35140_b200 import binding as tik
    tik.load()
    ok, hashes = audit.run_checks()
    assert ok
    path = os.path.join(os.path.dirname(audit.__file__), "audit_spec_b200.json")
    spec = json.load(open(path))
    recorded = spec["hashes"].get(tik.contract_id())
    if recorded is None:
        pytest.skip("no hashes recorded for contract %s" % tik.contract_id())
    assert hashes == recorded
