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


def both(ops, tensors, budget):
    """The oracle's plan, after checking that the library produces the same one."""
    want = po.generate(ops, tensors, budget)
    rc, actions, events, rep = api.plan_generate(ops, tensors, budget)
    assert (actions, events, rep.peak_bytes, rep.n_over_budget) == (want[0], want[1], want[2], want[4])
    assert abs(rep.overhead_seconds - want[3]) < 1e-12
    return want


def test_hand_case_skip_connection_locks_the_tensor_it_reads():
    """Four forward ops (op k reads tensor k-1, writes tensor k; op 3 also reads tensor 0: a skip connection),
    then backward ops 4..7 reading tensors 3, 2, 1, 0.  Every op 1 s, every tensor 100 B, budget 350.
    Ops 0-2 fill the pool to 300.  Op 3 allocates tensor 3: 300 + 100 >= 350.  Tensors 2, 0 (inputs) and 3 are
    locked, so tensor 1 is the only candidate -- without the skip connection it would have been tensor 0, whose
    reader is furthest away.  Next reader of tensor 1 = op 6: FLT = 3 s;
      MPS_compress = (100 - 25) * 3 / (0.5 + 0.5) = 225 > MPS_compute = 100 * 3 / 2 = 150  ->  compress.
    Pool 300 - 75 + 100 = 325 (the peak).  Ops 4, 5 free tensors 3, 2 (pool 125); op 6 decompresses tensor 1
    (125 + 100 < 350, no purge).  Overhead 0.5 + 0.5 = 1.0 s."""
    ops = [dict(time=1.0, inputs=[], outputs=[0]), dict(time=1.0, inputs=[0], outputs=[1]),
           dict(time=1.0, inputs=[1], outputs=[2]), dict(time=1.0, inputs=[2, 0], outputs=[3]),
           dict(time=1.0, inputs=[3], outputs=[]), dict(time=1.0, inputs=[2], outputs=[]),
           dict(time=1.0, inputs=[1], outputs=[]), dict(time=1.0, inputs=[0], outputs=[])]
    tensors = [T(100, 25, 0.5, 0.5, 2.0)] * 4
    actions, events, peak, overhead, over = both(ops, tensors, 350)
    assert actions == [po.KEEP, po.COMPRESS, po.KEEP, po.KEEP]
    assert events == [(3, 1, po.COMPRESS), (6, 1, po.KEEP)]
    assert (peak, overhead, over) == (325, 1.0, 0)
    # the same graph without the skip connection purges tensor 0 instead (FLT = 7 - 3 = 4 s, MPS 300)
    ops[3] = dict(time=1.0, inputs=[2], outputs=[3])
    actions, events, *_ = both(ops, tensors, 350)
    assert actions == [po.COMPRESS, po.KEEP, po.KEEP, po.KEEP] and events[0] == (3, 0, po.COMPRESS)


def test_hand_case_recovering_an_evicted_tensor_forces_another_purge():
    """Ops: 0 writes t0; 1 reads t0 writes t1; 2 reads t1 writes t2; 3 reads t2 and t0, writes t3 (10 B);
    4 reads t3 and t1.  t0, t1, t2 are 100 B; every op 1 s; budget 300.
    Op 2 allocates t2: pool 200 + 100 >= 300; t1, t2 locked, candidate t0 (next reader op 3, FLT 1 s):
      MPS_compute = 100 * 1 / 0.25 = 400 > MPS_compress = 75 * 1 / 1 = 75  ->  evict; pool 100 + 100 = 200.
    Op 3 needs t0 back: 200 + 100 >= 300 while t2, t0, t3 are locked; candidate t1 (cannot be recomputed,
    next reader op 4, FLT 1 s, MPS_compress 75) -> compressed: pool 200 - 75 = 125, then t0 is recomputed
    (pool 225) and t3 allocated (235, the peak).  t2 and t0 die after op 3 (pool 35); op 4 decompresses t1
    (35 + 100 < 300).  Overhead = recompute 0.25 + compress 0.5 + decompress 0.5 = 1.25 s."""
    ops = [dict(time=1.0, inputs=[], outputs=[0]), dict(time=1.0, inputs=[0], outputs=[1]),
           dict(time=1.0, inputs=[1], outputs=[2]), dict(time=1.0, inputs=[2, 0], outputs=[3]),
           dict(time=1.0, inputs=[3, 1], outputs=[])]
    tensors = [T(100, 25, 0.5, 0.5, 0.25), T(100, 25, 0.5, 0.5, -1.0), T(100, 25, 0.5, 0.5, 2.0), T(10, 10, 0.5, 0.5, 2.0)]
    actions, events, peak, overhead, over = both(ops, tensors, 300)
    assert actions == [po.EVICT, po.COMPRESS, po.KEEP, po.KEEP]
    assert events == [(2, 0, po.EVICT), (3, 1, po.COMPRESS), (3, 0, po.KEEP), (4, 1, po.KEEP)]
    assert (peak, overhead, over) == (235, 1.25, 0)


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
