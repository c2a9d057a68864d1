"""The ways a synchronous step can launch its boundary work (gp_config.overlap_slots).

With -2 the selection jobs, the decisions, the compaction and the merge of split outputs are one kernel behind the
attention kernel, whose jobs start when that kernel has reported their unit's summary logits complete; with -1 a
selection and a compaction kernel run one after the other (four launches); the default (0) picks between the two
by the pool's size, so the other tests of the synchronous mode run one or the other.  Here both are forced, and
the one kernel also runs beside the attention kernel on thread-block slots that kernel's grid gives up (N > 0).  Nothing about the results may change: the same lockstep comparison against the oracle
(actions, working-set sizes, Delta, retained sets, page tables, free list, summaries, attention outputs), over the
five configurations, the paper's page geometry, the Shrink policy, the entropy metric and RoPE, with slot counts
from one thread block to half the grid."""
import numpy as np
import pytest

from paper_2609_03494_b200 import binding as B
from paper_2609_03494_b200 import workload as W

from tests import lockstep as LS

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("slots", [64, -1, -2])
@pytest.mark.parametrize("config", [1, 2, 3, 4, 5])
def test_lockstep_configurations_with_overlapped_boundary_work(config, slots):
    st = LS.run_lockstep(W.parity_instance(config), overlap_slots=slots)
    assert st.decisions["act"] > 0 and st.near_ties == {"ws": 0, "sel": 0, "act": 0}


@pytest.mark.parametrize("slots", [1, 8, 148, 4000])
def test_slot_counts_from_one_block_to_half_the_grid(slots):
    st = LS.run_lockstep(W.parity_instance(1), overlap_slots=slots, tau=-0.05)
    assert st.actions.get(B.GP_ACT_GROW, 0) > 0 and st.actions.get(B.GP_ACT_COMPRESS, 0) > 0


@pytest.mark.parametrize("over", [dict(rope_theta=1e6, tau=-0.05), dict(policy=B.GP_POLICY_SHRINK, min_capacity=48, tau=-0.06,
                                                                       shrink_below=-0.085),
                                  dict(demand_metric=B.GP_METRIC_ENTROPY), dict(tau=-1.0)])
def test_variants_with_overlapped_boundary_work(over):
    st = LS.run_lockstep(W.parity_instance(1), overlap_slots=48, max_steps=200, **over)
    assert st.decisions["act"] > 0


def test_pages_of_256_tokens_with_overlapped_boundary_work():
    s = W.Shape(1, 8, 2, 64, page_size=256)
    reqs = [W.RequestSpec(i, p, 900, 0.05, share_group=-1) for i, p in enumerate((300, 40, 511))]
    wl = W.Workload("b256", 77, s, reqs, n_resident=3, initial_pages=0, max_pages_per_req=4, n_pages=14, k_loc=64)
    st = LS.run_lockstep(wl, tau=-0.05, summary_every=64, check_pool_every=32, overlap_slots=32)
    assert st.actions.get(B.GP_ACT_GROW, 0) >= 3 and st.decisions["sel"] > 0


@pytest.mark.parametrize("slots", [-1, -2])
@pytest.mark.parametrize("config,over", [(1, dict(tau=-0.05)), (3, dict()), (5, dict()),
                                         (5, dict(policy=B.GP_POLICY_SHRINK, min_capacity=64, tau=-0.03, shrink_below=-0.036))])
def test_compaction_that_claims_whole_units(config, over, slots):
    # with units for every thread block twice over the compaction claims a unit per ticket and moves its chunks in
    # order, without the per-chunk flags; forced here on small pools, with copy-on-write pages and Shrinks among them
    st = LS.run_lockstep(W.parity_instance(config), overlap_slots=slots, compact_by_unit=True, **over)
    assert st.decisions["sel"] > 0 and st.counters[8] > 0


def test_compaction_by_unit_with_pages_of_256_tokens():
    s = W.Shape(1, 8, 2, 64, page_size=256)
    reqs = [W.RequestSpec(i, p, 900, 0.05, share_group=-1) for i, p in enumerate((300, 40, 511))]
    wl = W.Workload("b256", 77, s, reqs, n_resident=3, initial_pages=0, max_pages_per_req=4, n_pages=14, k_loc=64)
    st = LS.run_lockstep(wl, tau=-0.05, summary_every=64, check_pool_every=32, compact_by_unit=True)
    assert st.actions.get(B.GP_ACT_COMPRESS, 0) + st.actions.get(B.GP_ACT_COMPRESS_FALLBACK, 0) >= 3


def test_compaction_by_unit_in_the_asynchronous_mode():
    st = LS.run_lockstep(W.parity_instance(1), async_boundary=True, compact_by_unit=True, tau=-0.05)
    assert st.decisions["sel"] > 0 and st.counters[8] > 0
    st = LS.run_lockstep(W.parity_instance(5), async_boundary=True, compact_by_unit=True)
    assert st.decisions["sel"] > 0 and st.counters[4] > 0          # copy-on-write pages among them
