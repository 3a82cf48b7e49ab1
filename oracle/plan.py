"""Plan generation, Algorithm 1 with the MPS metric (Eq. 5) -- oracle.

THIS IS TEST INFRASTRUCTURE: a plain, slow restatement of the paper's plan-generation mechanism used only
to check the library's fh_plan_generate.  It shares no code with it.

Algorithm 1 (Plan Generation Mechanism): Main walks the computation sequence; Compute(op) gives every
COMPRESSED input its dense buffer back and recovers every EVICTED one, then allocates the outputs; Alloc
purges while pool_size + size >= memory_budget: the tensor with the largest MPS is evicted when its
MPS_compute exceeds its MPS_compress, compressed otherwise.
Eq. 5: RW(d) = SM(d) * FLT(d), MPS(d) = RW(d) / (PC(d) + RC(d)); Eq. 6 (the recomputation cost) is an input.

Readings where the paper is silent (the same as the library documents): the current op's tensors are
locked; a tensor leaves the pool after its last reader; tensors nothing produces are resident from the
start; candidates are resident tensors with a later reader; ties go to the lower index; FLT is measured
from the start of the current op to the start of the next reader; a technique that cannot apply has MPS 0;
if nothing can be purged the allocation goes over budget and is counted.
"""
from fractions import Fraction

KEEP, COMPRESS, EVICT = 0, 1, 2


def generate(ops, tensors, memory_budget):
    """ops: list of dicts {time, inputs, outputs}; tensors: list of dicts {bytes, packed_bytes, t_compress,
    t_decompress, t_recompute}.  Returns (actions, events, peak_bytes, overhead_seconds, n_over_budget)."""
    nT = len(tensors)
    start = [0.0]
    for op in ops:
        start.append(start[-1] + op["time"])
    readers = [[i for i, op in enumerate(ops) if t in op["inputs"]] for t in range(nT)]
    produced = [any(t in op["outputs"] for op in ops) for t in range(nT)]
    state = ["none"] * nT
    pool = 0
    for t in range(nT):
        if not produced[t] and readers[t]:
            state[t] = "resident"
            pool += tensors[t]["bytes"]
    peak, overhead, n_over = pool, 0.0, 0
    actions, events = [KEEP] * nT, []

    def next_reader(t, i):
        later = [r for r in readers[t] if r > i]
        return later[0] if later else None

    def mps(t, i):
        d = tensors[t]
        flt = start[next_reader(t, i)] - start[i]
        compress = (d["bytes"] - d["packed_bytes"]) * flt / (d["t_compress"] + d["t_decompress"]) \
            if d["packed_bytes"] < d["bytes"] else 0.0
        compute = d["bytes"] * flt / d["t_recompute"] if d["t_recompute"] >= 0 else 0.0
        return compute, compress

    for i, op in enumerate(ops):
        locked = set(op["inputs"]) | set(op["outputs"])

        def alloc(size):
            nonlocal pool, peak, overhead, n_over
            while pool + size >= memory_budget:
                best, best_val = None, 0.0
                for t in range(nT):
                    if state[t] != "resident" or t in locked or next_reader(t, i) is None:
                        continue
                    compute, compress = mps(t, i)
                    if max(compute, compress) > best_val:
                        best, best_val = t, max(compute, compress)
                if best is None:
                    n_over += 1
                    break
                compute, compress = mps(best, i)
                d = tensors[best]
                if compute > compress:
                    state[best] = "evicted"
                    pool -= d["bytes"]
                    actions[best] = EVICT
                    events.append((i, best, EVICT))
                else:
                    state[best] = "compressed"
                    pool -= d["bytes"] - d["packed_bytes"]
                    overhead += d["t_compress"]
                    actions[best] = COMPRESS
                    events.append((i, best, COMPRESS))
            pool += size
            peak = max(peak, pool)

        for t in op["inputs"]:
            d = tensors[t]
            if state[t] == "compressed":
                alloc(d["bytes"])
                pool -= d["packed_bytes"]
                overhead += d["t_decompress"]
                state[t] = "resident"
                events.append((i, t, KEEP))
            elif state[t] == "evicted":
                alloc(d["bytes"])
                overhead += d["t_recompute"]
                state[t] = "resident"
                events.append((i, t, KEEP))
        for t in op["outputs"]:
            if state[t] == "none":
                alloc(tensors[t]["bytes"])
                state[t] = "resident"
        for t in list(op["inputs"]) + list(op["outputs"]):
            if state[t] == "resident" and next_reader(t, i) is None:
                state[t] = "dead"
                pool -= tensors[t]["bytes"]
    return actions, events, peak, overhead, n_over
