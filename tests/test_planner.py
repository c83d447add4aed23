"""The host planner's choices for every configured layer, pinned (CPU only).

ssconv_plan_for_sms is host arithmetic: tile width, K split, thread blocks and pairing for a device
with the given number of SMs.  The table below is the planner's answer for 148 SMs on the layers of
the four workload configurations; a change of one of its cost constants shows up here as a diff that
has to be looked at (and re-measured) rather than slipping through.  Regenerate with
    python -m tests.test_planner
"""
import json
import os

import pytest

from paper_2411_00288_b200 import api, build as libbuild, synth

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "planner_148sm.json")
SMS = 148


def _plans():
    libbuild.build()
    out = {}
    for cfg in (2, 3, 4, 5):
        for spec in synth.config_layers(cfg):
            desc = api.desc_from_spec(spec)
            row = {}
            for sparse in (True, False):
                p = api.ssconv_plan_for_sms(desc, sparse, SMS)
                row["sparse" if sparse else "dense"] = [p["tile_positions"], int(p["split"]), int(p["pair"]), p["ctas"]]
            out[f"cfg{cfg}:{spec.name}"] = row
    return out


def test_planner_choices_match_the_pinned_table():
    with open(GOLDEN) as f:
        want = json.load(f)
    got = _plans()
    assert set(got) == set(want)
    diff = {k: (want[k], got[k]) for k in got if got[k] != want[k]}
    assert not diff, f"planner choices changed (pinned, now): {diff}"


def test_planner_invariants():
    for name, row in _plans().items():
        for kind, (bn, split, pair, ctas) in row.items():
            assert 48 <= bn <= 240 and bn % 16 == 0, (name, kind, bn)
            assert 1 <= ctas <= SMS
            assert not (split and pair)
            if pair:
                assert ctas % 2 == 0


def test_never_more_blocks_than_sms_and_scaling_with_the_sm_count():
    spec = synth.config_layers(3)[4]
    desc = api.desc_from_spec(spec)
    for sms in (1, 2, 16, 74, 132, 148, 160):
        p = api.ssconv_plan_for_sms(desc, True, sms)
        assert 1 <= p["ctas"] <= sms


def test_window_extent_is_the_output_extent_formula():
    for cfg in (1, 2, 3, 4, 5):
        for s in synth.config_layers(cfg):
            assert api.ssconv_window_extent(s.H, s.KH, s.stride, s.pad, s.dil) == s.H_out
    assert api.ssconv_window_extent(5, 7, 1, 0, 1) == 0          # the window does not fit
    assert api.ssconv_window_extent(112, 3, 2, 1, 1) == 56       # the stack's max-pool


if __name__ == "__main__":
    os.makedirs(os.path.dirname(GOLDEN), exist_ok=True)
    with open(GOLDEN, "w") as f:
        json.dump(_plans(), f, indent=0, sort_keys=True)
    print("wrote", GOLDEN)
