"""Plan generation (Algorithm 1, Eq. 5): the oracle against hand-worked cases, the library against the
oracle.  Host-only: no GPU needed."""
import numpy as np
import pytest

from oracle import plan as po
from paper_2510_11400_b200 import api, build


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    api.lib()


def T(bytes_, packed, tc, td, tr):
    return dict(bytes=bytes_, packed_bytes=packed, t_compress=tc, t_decompress=td, t_recompute=tr)


def chain(n, op_time=1.0):
    """Forward ops 0..n-1 (op k reads tensor k-1, writes tensor k), then backward ops that read the saved
    tensors in reverse order: the shape of one training step."""
    ops = [dict(time=op_time, inputs=[k - 1] if k else [], outputs=[k]) for k in range(n)]
    ops += [dict(time=op_time, inputs=[k], outputs=[]) for k in reversed(range(n))]
    return ops


def test_hand_case_mps_values_and_choice():
    """Three forward ops and the three backward ops reading their outputs in reverse; every tensor 100 B.
    Budget 250: allocating tensor 2 (op 2) meets pool 200 + 100 >= 250.  Tensor 1 is locked (input of op 2),
    so tensor 0 is the only candidate: next reader = op 5, FLT = 5 - 2 = 3 s.
      MPS_compress = (100 - 25) * 3 / (0.5 + 0.5) = 225;  MPS_compute = 100 * 3 / 2 = 150  ->  compress.
    Pool 200 - 75 + 100 = 225.  Backward: op 3 reads 2, op 4 reads 1, op 5 reads 0: decompress at op 5 needs
    100 more while only 25 is held -> 25 + 100 < 250, no purge.  Overhead 0.5 + 0.5 = 1.0 s, peak 225."""
    ops = chain(3)
    tensors = [T(100, 25, 0.5, 0.5, 2.0)] * 3
    actions, events, peak, overhead, over = po.generate(ops, tensors, 250)
    assert actions == [po.COMPRESS, po.KEEP, po.KEEP]
    assert events == [(2, 0, po.COMPRESS), (5, 0, po.KEEP)]
    assert (peak, overhead, over) == (225, 1.0, 0)
    # a cheap recomputation flips the choice: MPS_compute = 100 * 3 / 0.5 = 600 > 225 -> evict
    tensors = [T(100, 25, 0.5, 0.5, 0.5)] * 3
    actions, events, peak, overhead, over = po.generate(ops, tensors, 250)
    assert actions == [po.EVICT, po.KEEP, po.KEEP] and events[0] == (2, 0, po.EVICT)
    assert (peak, overhead) == (200, 0.5)


def test_large_budget_changes_nothing_and_small_budget_is_reported():
    ops = chain(4)
    tensors = [T(100, 25, 0.5, 0.5, 2.0)] * 4
    actions, events, peak, overhead, over = po.generate(ops, tensors, 10_000)
    assert actions == [po.KEEP] * 4 and events == [] and overhead == 0.0 and peak == 400 and over == 0
    # a budget below two live tensors cannot be met: locked tensors are never purged
    actions, events, peak, overhead, over = po.generate(ops, tensors, 150)
    assert over > 0


def test_longer_freed_lifetime_wins():
    """Equal sizes and costs: the tensor whose next reader is furthest away has the largest MPS (Eq. 5's FLT)."""
    ops = chain(5)
    tensors = [T(100, 25, 0.5, 0.5, -1.0)] * 5
    actions, events, *_ = po.generate(ops, tensors, 450)
    purged = [e for e in events if e[2] == po.COMPRESS]
    assert purged[0][1] == 0          # tensor 0 is read last in the backward pass


def random_graph(rng, n):
    ops = chain(n, op_time=1.0)
    for op in ops:
        op["time"] = float(rng.integers(1, 8)) / 4.0
    tensors = []
    for _ in range(n):
        b = int(rng.integers(1, 64)) * 256
        packed = int(b * rng.choice([0.07, 0.13, 0.26, 0.6, 1.0]))
        tensors.append(T(b, packed, float(rng.integers(1, 16)) / 64.0, float(rng.integers(1, 16)) / 64.0,
                         float(rng.choice([-1.0, 0.25, 1.0, 4.0]))))
    # some skip connections
    for _ in range(n // 3):
        a, b = sorted(rng.integers(0, n, 2))
        if a != b and int(a) not in ops[int(b)]["inputs"]:
            ops[int(b)]["inputs"].append(int(a))
    return ops, tensors


@pytest.mark.parametrize("seed", range(12))
def test_library_agrees_with_the_oracle_on_random_graphs(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(4, 24))
    ops, tensors = random_graph(rng, n)
    total = sum(t["bytes"] for t in tensors)
    for frac in (2.0, 0.7, 0.45, 0.25):
        budget = int(total * frac)
        want = po.generate(ops, tensors, budget)
        rc, actions, events, rep = api.plan_generate(ops, tensors, budget)
        assert actions == want[0]
        assert events == want[1]
        assert rep.peak_bytes == want[2] and rep.n_over_budget == want[4]
        assert abs(rep.overhead_seconds - want[3]) < 1e-12
        assert rc == (api.FH_ERR_CAPACITY if want[4] else api.FH_OK)
        # invariants of a plan: whatever was purged and is read later comes back before that reader
        held = {}
        for op, t, kind in events:
            if kind in (po.COMPRESS, po.EVICT):
                held[t] = op
            else:
                assert t in held and held.pop(t) <= op
        if not want[4]:
            assert rep.peak_bytes < budget


def test_argument_errors():
    ops = chain(2)
    tensors = [T(100, 25, 0.5, 0.5, 2.0)] * 2
    assert api.plan_generate(ops, [T(100, 25, 0.0, 0.0, 2.0)] * 2, 100)[0] == api.FH_ERR_ARG     # free compression: MPS undefined
    assert api.plan_generate(ops, [T(100, 25, 0.5, 0.5, 0.0)] * 2, 100)[0] == api.FH_ERR_ARG     # free recomputation
    bad = [dict(time=1.0, inputs=[5], outputs=[0])]
    assert api.plan_generate(bad, tensors, 100)[0] == api.FH_ERR_ARG
