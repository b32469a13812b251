"""Full traces of the large configurations through the library's bookkeeping on the CPU, every
output of every request against the oracle.  Marked ``slow`` (a minute or two each); they are
still part of the default CPU run."""
import pytest

from full_trace_util import compare_full_trace

pytestmark = pytest.mark.slow


@pytest.fixture(scope="module")
def eakv():
    from paper_2609_33762_b200 import build, eakv as m
    build.build()
    return m


def test_config4_full_trace_smallest_tier(eakv):
    """All 7,680 requests (23.8 M block references) of config 4 at the 64 GiB end of its sweep,
    through the single calls: nothing survives between turns (working set 1.5 TiB)."""
    out = compare_full_trace(eakv, "c4", 64)
    assert out["requests"] == 7680 and out["references"] == 23810566
    assert out["restored_blocks"] == 0 and out["computed_prefill"] == 697212521


def test_config4_full_trace_largest_tier_through_the_turn_engine(eakv):
    """The 512 GiB end through eakv_turn_begin / eakv_turn_end, compared per request (view
    scalars and arrays), not through totals."""
    out = compare_full_trace(eakv, "c4", 512, turn_engine=True)
    assert out["requests"] == 7680 and out["restored_blocks"] > 7_000_000
    assert out["computed_prefill"] == 469895177


def test_config3_full_trace_conditioned_through_the_turn_engine(eakv):
    out = compare_full_trace(eakv, "c3", 32, policy=2, turn_engine=True)
    assert out["requests"] == 1280 and out["stored_blocks"] < out["restored_blocks"]
