"""L2 residency of a state array (kv_set_l2_residency): an access-policy window on the touch
counts, or on the pair bytes when the counts exceed the budget, changes where lines live in
the cache and nothing else -- every result stays bit for bit the oracle's."""
import pytest

from paper_2604_26968_b200 import binding as B
from paper_2604_26968_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("budget", [48 << 20, 1 << 20, 64 << 10])
def test_results_do_not_depend_on_the_window(fused, budget):
    """Pool 2 at 1/16: 196,608 entries = 768 KB of touch counts, 192 KB of pair bytes: the three
    budgets give a window on the whole touch array, on the whole pair array, on a third of it."""
    from lockstep import Lockstep
    w = W.config(2, scale=1 / 16)
    ls = Lockstep(w, payload=False, batch_bytes=8 << 20, fused=fused, l2_budget=budget)
    for e in range(4):
        ls.epoch(e)
    assert ls.gpu.pool.kv_set_l2_residency(0) == B.KV_OK       # and off again
    ls.epoch(4)
    ls.close()


def test_mixed_pool_with_block_selection_and_the_multi_launch_selection():
    from lockstep import Lockstep
    w = W.config(5, scale=1 / 128)
    for p in w.parts:
        p.ring_slots = w.k + 64
    ls = Lockstep(w, payload=True, batch_bytes=1 << 20, fused=True, counted=True, l2_budget=256 << 10,
                  select_variant=0)
    for e in range(3):
        ls.epoch(e)
    ls.epoch(3, k_blocks=40)
    ls.close()
