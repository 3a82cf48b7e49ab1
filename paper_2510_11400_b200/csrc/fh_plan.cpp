// Plan generation (Algorithm 1, MPS metric of Eq. 5): host-only part of the C ABI in include/fh.h.
#include "../../include/fh.h"

#include <algorithm>
#include <vector>

namespace {

enum State { kNone = 0, kResident, kCompressed, kEvicted, kDead };

struct Planner {
  const fh_plan_op* ops;
  int32_t n_ops;
  const fh_plan_tensor* tensors;
  int32_t n_tensors;
  uint64_t budget;
  std::vector<int> state;
  std::vector<std::vector<int32_t>> readers;  // per tensor: ops that read it, ascending
  std::vector<double> start;                  // start time of every op
  std::vector<char> locked;
  uint64_t pool = 0, peak = 0;
  double overhead = 0.0;
  int32_t n_events = 0, n_over = 0;
  int32_t* actions;
  fh_plan_event* events;
  int32_t max_events;

  void note(int32_t op, int32_t t, int32_t kind) {
    if (events && n_events < max_events) events[n_events] = fh_plan_event{op, t, kind};
    ++n_events;
  }
  // first op after `op` that reads tensor t, or -1
  int32_t next_reader(int32_t t, int32_t op) const {
    const auto& r = readers[t];
    auto it = std::upper_bound(r.begin(), r.end(), op);
    return it == r.end() ? -1 : *it;
  }
  // Alloc: purge by largest MPS until the request fits
  void alloc(int32_t op, uint64_t size) {
    while (pool + size >= budget) {
      int32_t best = -1;
      double best_mps = 0.0, best_compute = 0.0, best_compress = 0.0;
      for (int32_t t = 0; t < n_tensors; ++t) {
        if (state[t] != kResident || locked[t]) continue;
        const int32_t nr = next_reader(t, op);
        if (nr < 0) continue;
        const fh_plan_tensor& d = tensors[t];
        const double flt = start[nr] - start[op];
        double mps_compress = 0.0, mps_compute = 0.0;
        if (d.packed_bytes < d.bytes) mps_compress = (double)(d.bytes - d.packed_bytes) * flt / (d.t_compress + d.t_decompress);
        if (d.t_recompute >= 0.0) mps_compute = (double)d.bytes * flt / d.t_recompute;
        const double mps = std::max(mps_compress, mps_compute);
        if (mps > best_mps) {
          best = t;
          best_mps = mps;
          best_compute = mps_compute;
          best_compress = mps_compress;
        }
      }
      if (best < 0) {  // nothing left to purge
        ++n_over;
        break;
      }
      const fh_plan_tensor& d = tensors[best];
      if (best_compute > best_compress) {
        state[best] = kEvicted;
        pool -= d.bytes;
        actions[best] = FH_EVICT;
        note(op, best, FH_EVICT);
      } else {
        state[best] = kCompressed;
        pool -= d.bytes - d.packed_bytes;
        overhead += d.t_compress;
        actions[best] = FH_COMPRESS;
        note(op, best, FH_COMPRESS);
      }
    }
    pool += size;
    peak = std::max(peak, pool);
  }
  // Compute: inputs back in memory, outputs allocated
  void compute(int32_t i) {
    const fh_plan_op& op = ops[i];
    for (int32_t k = 0; k < op.n_inputs; ++k) locked[op.inputs[k]] = 1;
    for (int32_t k = 0; k < op.n_outputs; ++k) locked[op.outputs[k]] = 1;
    for (int32_t k = 0; k < op.n_inputs; ++k) {
      const int32_t t = op.inputs[k];
      const fh_plan_tensor& d = tensors[t];
      if (state[t] == kCompressed) {
        alloc(i, d.bytes);
        pool -= d.packed_bytes;  // the packed copy is released once the dense one is back
        overhead += d.t_decompress;
        state[t] = kResident;
        note(i, t, FH_KEEP);
      } else if (state[t] == kEvicted) {
        alloc(i, d.bytes);
        overhead += d.t_recompute;
        state[t] = kResident;
        note(i, t, FH_KEEP);
      }
    }
    for (int32_t k = 0; k < op.n_outputs; ++k) {
      const int32_t t = op.outputs[k];
      if (state[t] == kNone) {
        alloc(i, tensors[t].bytes);
        state[t] = kResident;
      }
    }
    for (int32_t k = 0; k < op.n_inputs; ++k) locked[op.inputs[k]] = 0;
    for (int32_t k = 0; k < op.n_outputs; ++k) locked[op.outputs[k]] = 0;
    // tensors nobody reads any more leave the pool
    for (int32_t k = 0; k < op.n_inputs + op.n_outputs; ++k) {
      const int32_t t = k < op.n_inputs ? op.inputs[k] : op.outputs[k - op.n_inputs];
      if (state[t] == kResident && next_reader(t, i) < 0) {
        state[t] = kDead;
        pool -= tensors[t].bytes;
      }
    }
  }
};

}  // namespace

extern "C" int fh_plan_generate(const fh_plan_op* ops, int32_t n_ops, const fh_plan_tensor* tensors, int32_t n_tensors,
                                uint64_t memory_budget, int32_t* actions, fh_plan_event* events, int32_t max_events,
                                fh_plan_report* report) {
  if (!ops || !tensors || !actions || !report || n_ops < 0 || n_tensors < 0 || max_events < 0) return FH_ERR_ARG;
  for (int32_t t = 0; t < n_tensors; ++t) {
    const fh_plan_tensor& d = tensors[t];
    if (!(d.t_compress >= 0.0) || !(d.t_decompress >= 0.0)) return FH_ERR_ARG;
    if (d.packed_bytes < d.bytes && !(d.t_compress + d.t_decompress > 0.0)) return FH_ERR_ARG;
    if (d.t_recompute == 0.0) return FH_ERR_ARG;
  }
  Planner p;
  p.ops = ops;
  p.n_ops = n_ops;
  p.tensors = tensors;
  p.n_tensors = n_tensors;
  p.budget = memory_budget;
  p.actions = actions;
  p.events = events;
  p.max_events = max_events;
  p.state.assign(n_tensors, kNone);
  p.readers.assign(n_tensors, {});
  p.locked.assign(n_tensors, 0);
  p.start.assign((size_t)n_ops + 1, 0.0);
  std::vector<char> produced(n_tensors, 0);
  for (int32_t i = 0; i < n_ops; ++i) {
    const fh_plan_op& op = ops[i];
    if (!(op.time >= 0.0) || op.n_inputs < 0 || op.n_outputs < 0 || (op.n_inputs && !op.inputs) ||
        (op.n_outputs && !op.outputs))
      return FH_ERR_ARG;
    p.start[i + 1] = p.start[i] + op.time;
    for (int32_t k = 0; k < op.n_inputs; ++k) {
      if (op.inputs[k] < 0 || op.inputs[k] >= n_tensors) return FH_ERR_ARG;
      if (p.readers[op.inputs[k]].empty() || p.readers[op.inputs[k]].back() != i) p.readers[op.inputs[k]].push_back(i);
    }
    for (int32_t k = 0; k < op.n_outputs; ++k) {
      if (op.outputs[k] < 0 || op.outputs[k] >= n_tensors) return FH_ERR_ARG;
      produced[op.outputs[k]] = 1;
    }
  }
  for (int32_t t = 0; t < n_tensors; ++t) {
    actions[t] = FH_KEEP;
    if (!produced[t] && !p.readers[t].empty()) {  // graph inputs: resident from the start
      p.state[t] = kResident;
      p.pool += tensors[t].bytes;
    }
  }
  p.peak = p.pool;
  for (int32_t i = 0; i < n_ops; ++i) p.compute(i);  // Main
  report->peak_bytes = p.peak;
  report->overhead_seconds = p.overhead;
  report->n_events = p.n_events;
  report->n_over_budget = p.n_over;
  return p.n_over ? FH_ERR_CAPACITY : FH_OK;
}
