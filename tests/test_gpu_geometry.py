"""The paper's page geometry (Sec. 5.1, App. B.2, App. D.1): pages of 256 tokens, a protected window of 16, a local
quota of 64.  Capacity grows by a page of 256 slots, the working sets of Eq. 7 leave out the newest page, the
candidates of Eq. 10 only the 16 protected tokens, blocks for the local quota are the 256-token pages (the last
one short), and a compression frees exactly one page worth of slots.  On the GPU a page of the method is a group
of 16-token tiles; the comparison with the oracle is the usual lockstep one, every decision included.  Smaller
pages (32, 64 tokens) go through the same code with more boundaries per step run."""
import numpy as np
import pytest

from paper_2609_03494_b200 import binding as B
from paper_2609_03494_b200 import workload as W
from tests import lockstep as LS

pytestmark = pytest.mark.gpu
NO_NEAR_TIES = {"ws": 0, "sel": 0, "act": 0}


def _report(name, st):
    print(f"\n[geometry {name}] steps {st.steps} tokens {st.tokens} attn max {st.attn_max_abs:.2e} decisions {st.decisions} "
          f"near-ties {st.near_ties} actions {st.actions} cow {st.counters[4]}")


def _workload(b, prompts, n_steps, cap, n_pages, shape=(1, 8, 2, 64), groups=None, k_loc=None, initial_pages=0):
    s = W.Shape(*shape, page_size=b)
    reqs = [W.RequestSpec(i, p, n_steps, 0.05, share_group=-1 if groups is None else groups[i]) for i, p in enumerate(prompts)]
    return W.Workload(f"b{b}", 77, s, reqs, n_resident=len(reqs), initial_pages=initial_pages, max_pages_per_req=cap,
                      n_pages=n_pages, k_loc=b // 4 if k_loc is None else k_loc)


def test_paper_defaults_256_16_64():
    # three requests; 900 steps take them over three or four boundaries each: grants up to the cap of four pages,
    # then compressions that free 256 slots each
    wl = _workload(256, (300, 40, 511), 900, cap=4, n_pages=14)
    st = LS.run_lockstep(wl, tau=-0.05, summary_every=64, check_pool_every=32)
    _report("256/16/64", st)
    assert st.actions.get(B.GP_ACT_GROW, 0) >= 3 and st.actions.get(B.GP_ACT_COMPRESS, 0) + st.actions.get(B.GP_ACT_COMPRESS_FALLBACK, 0) >= 3
    assert st.decisions["sel"] > 0 and st.near_ties == NO_NEAR_TIES


def test_paper_defaults_on_the_8b_head_shape_with_rope():
    wl = _workload(256, (500, 250), 560, cap=3, n_pages=8, shape=(2, 32, 8, 128))
    st = LS.run_lockstep(wl, tau=-0.02, rope_theta=1e6, summary_every=64, check_pool_every=64)
    _report("256 8B shape", st)
    assert st.decisions["act"] >= 3 and st.decisions["sel"] > 0


@pytest.mark.parametrize("b,over", [(32, dict(tau=-1.0, n_pages=11)), (64, dict(tau=-0.03)), (128, dict(tau=0.0, k_loc=0)),
                                   (64, dict(async_boundary=True, tau=-0.03)),
                                   (64, dict(policy=B.GP_POLICY_SHRINK, shrink_below=0.0, min_capacity=128, tau=0.05))])
def test_other_page_sizes_grants_fallbacks_stalls_async_and_shrink(b, over):
    wl = _workload(b, (3 * b - 5, 17, 2 * b + 9, b), 8 * b, cap=6, n_pages=20, k_loc=over.pop("k_loc", None))
    st = LS.run_lockstep(wl, **over)
    _report(f"b={b} {over}", st)
    assert st.decisions["act"] > 8
    if over.get("n_pages") == 11:
        assert st.actions.get(B.GP_ACT_COMPRESS_FALLBACK, 0) > 0          # the pool ran dry: asked to grow, compressed
    if over.get("policy") == B.GP_POLICY_SHRINK:
        assert st.actions.get(B.GP_ACT_SHRINK, 0) > 0 and st.counters[10] > 0


def test_shared_prompt_pages_of_64_tokens_are_copied_before_the_first_compaction():
    # two groups of three on a shared 192-token prompt (three pages of 64 tokens = twelve tiles each), ten decode pages
    b = 64
    wl = _workload(b, (192,) * 6, 4 * b, cap=6, n_pages=2 * 3 + 6 * 4, groups=(0, 0, 0, 1, 1, 1), initial_pages=4)
    st = LS.run_lockstep(wl, tau=0.0)
    _report("b=64 shared", st)
    assert st.counters[4] > 0                                         # copy-on-write happened, counted in pages of the method
    assert st.actions.get(B.GP_ACT_COMPRESS, 0) > 0
