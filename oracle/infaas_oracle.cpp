// CPU oracle for batched model-variant selection and per-variant load tallies.
//
// TEST INFRASTRUCTURE ONLY.  This file is the plain, slow reference that the CUDA path is
// compared against.  It shares no code, header, table or helper with the CUDA path and is
// never called by it.  Only the tests, the smoke check and the benchmark's CPU-baseline
// leg may build or call it.
//
// What it computes, and where the paper states it:
//   * The query is (application/task, latency requirement, accuracy requirement) and the
//     answer is one variant of that task that meets both (Section 3.1, Table 4; Section 4.1,
//     "Case I: on arrival of a query").
//   * Among the variants that meet the requirements the cheapest one is wanted (Section 2.2,
//     the worked example around Table 2 / Table 3: at a 300 ms SLO the cost-1 variant wins,
//     at 50 ms the cost-3 variant).
//   * Static profiles are not enough: a variant that is already busy serves later, so its
//     expected latency grows with its load (Section 4, the list of dynamic aspects).
//   * When nothing meets the requirements, a variant that comes closest in accuracy and/or
//     latency is suggested (Section 4.1, last sentence of the first paragraph).
//   * Load per variant is tracked from the queries it serves and its batch size, and is
//     refreshed periodically (Section 4.2.2, scaling-up algorithm; Section 5).
//
// Everything is brute force over the full, unsorted, unpruned catalog.  There is no
// sorting, no pruning, no early exit and no blocking.  Readings of points the paper leaves
// open (ties, the queueing term, the distance used for "closest", the queue recursion) are
// this build's choices; those constants are "parity unpinned" by the paper itself, the
// structure around them is pinned by the tests under tests/ (worked example of Table 2,
// brute-force enumeration, closed forms, exact-rational ordering).
//
// Arithmetic: unsigned integers only.  Latency in microseconds (u32), accuracy in basis
// points (u16), cost in integer units (u32).

#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>

namespace {

struct Row {              // 24 bytes, same field order as the public catalog row
  uint16_t task;
  uint16_t arch;
  uint8_t hw;
  uint8_t opt;
  uint16_t batch;
  uint32_t lat_us;
  uint16_t acc_bp;
  uint16_t reserved;
  uint32_t cost;
  uint32_t queued;
};
static_assert(sizeof(Row) == 24, "row layout");

const uint64_t U32_MAX = 0xFFFFFFFFull;
const uint32_t NO_FEASIBLE_BIT = 0x80000000u;
const uint32_t INVALID = 0xFFFFFFFFu;

// Predicted latency of a variant that already has `queued` queries waiting: its own batch
// latency plus the time to work off the queue, batch by batch, as a single floor division
// of the product.  Saturates at 2^32-1.
uint32_t pred_lat(uint32_t lat_us, uint32_t queued, uint16_t batch) {
  uint64_t wait = (uint64_t)queued * (uint64_t)lat_us / (uint64_t)batch;
  uint64_t p = (uint64_t)lat_us + wait;
  return (uint32_t)(p > U32_MAX ? U32_MAX : p);
}

// Lexicographic "a < b" on (k0, k1, k2, k3, k4).
struct Key {
  uint64_t k[5];
};
bool key_less(const Key &a, const Key &b) {
  for (int i = 0; i < 5; ++i) {
    if (a.k[i] < b.k[i]) return true;
    if (a.k[i] > b.k[i]) return false;
  }
  return false;
}

// One query against the variants of its task.
//   feasible(v)  <=>  pred(v) <= slo  and  acc(v) >= min_acc
//   if some variant is feasible: the feasible variant with the smallest
//       (cost, pred, 10000-acc, id)
//   else: bit 31 set, low bits = variant with the smallest
//       (d, cost, pred, 10000-acc, id),  d = 10000*max(0,pred-slo) + slo*max(0,min_acc-acc)
uint32_t select_one(const Row *rows, const uint32_t *queued, const std::vector<uint32_t> &members,
                    uint32_t slo, uint16_t min_acc) {
  if (members.empty()) return INVALID;
  bool have_feasible = false, have_any = false;
  Key best_f{}, best_m{};
  uint32_t arg_f = 0, arg_m = 0;
  for (uint32_t v : members) {
    const Row &r = rows[v];
    uint32_t p = pred_lat(r.lat_us, queued[v], r.batch);
    bool ok = (p <= slo) && (r.acc_bp >= min_acc);
    uint64_t inv_acc = (uint64_t)(10000 - (int)r.acc_bp);
    if (ok) {
      Key k{{0, r.cost, p, inv_acc, v}};
      if (!have_feasible || key_less(k, best_f)) {
        best_f = k;
        arg_f = v;
        have_feasible = true;
      }
    }
    uint64_t over_lat = p > slo ? (uint64_t)(p - slo) : 0;
    uint64_t under_acc = min_acc > r.acc_bp ? (uint64_t)(min_acc - r.acc_bp) : 0;
    uint64_t d = 10000ull * over_lat + (uint64_t)slo * under_acc;
    Key k{{d, r.cost, p, inv_acc, v}};
    if (!have_any || key_less(k, best_m)) {
      best_m = k;
      arg_m = v;
      have_any = true;
    }
  }
  return have_feasible ? arg_f : (NO_FEASIBLE_BIT | arg_m);
}

std::vector<std::vector<uint32_t>> members_by_task(const Row *rows, uint32_t n_variants,
                                                   uint32_t n_tasks) {
  std::vector<std::vector<uint32_t>> m(n_tasks);
  for (uint32_t v = 0; v < n_variants; ++v)
    if (rows[v].task < n_tasks) m[rows[v].task].push_back(v);
  return m;
}

}  // namespace

extern "C" {

uint32_t oracle_pred_lat(uint32_t lat_us, uint32_t queued, uint16_t batch) {
  return pred_lat(lat_us, queued, batch);
}

// Decide every query against one load snapshot (`queued`, one entry per variant).
// `n_threads` only splits the query range; each query is decided independently.
void oracle_select(const void *rows_v, uint32_t n_variants, uint32_t n_tasks,
                   const uint32_t *queued, const uint16_t *task, const uint32_t *slo_us,
                   const uint16_t *min_acc_bp, uint64_t n, uint32_t *decision, int n_threads) {
  const Row *rows = (const Row *)rows_v;
  auto members = members_by_task(rows, n_variants, n_tasks);
  auto work = [&](uint64_t lo, uint64_t hi) {
    for (uint64_t q = lo; q < hi; ++q) {
      if (task[q] >= n_tasks) {
        decision[q] = INVALID;
        continue;
      }
      decision[q] = select_one(rows, queued, members[task[q]], slo_us[q], min_acc_bp[q]);
    }
  };
  if (n_threads <= 1) {
    work(0, n);
    return;
  }
  std::vector<std::thread> th;
  for (int i = 0; i < n_threads; ++i)
    th.emplace_back(work, n * (uint64_t)i / n_threads, n * (uint64_t)(i + 1) / n_threads);
  for (auto &t : th) t.join();
}

// End of a window: tally the window's feasible decisions per variant, then let every
// variant's queue take the arrivals and drain at its saturation rate for `window_us`.
//   count(v)  = number of decisions equal to v (bit 31 clear, v < n_variants)
//   drain(v)  = min(2^32-1, floor(window_us * batch / lat_us))
//   queued(v) = max(0, min(2^32-1, queued + count) - drain)
// counters[0..2] += (feasible decisions tallied, NO_FEASIBLE decisions, invalid decisions).
void oracle_load_update(const void *rows_v, uint32_t n_variants, uint32_t *queued,
                        uint64_t *served_total, uint64_t counters[3], const uint32_t *decision,
                        uint64_t n, uint32_t window_us) {
  const Row *rows = (const Row *)rows_v;
  std::vector<uint64_t> count(n_variants, 0);
  for (uint64_t q = 0; q < n; ++q) {
    uint32_t d = decision[q];
    if (d == INVALID) {
      counters[2] += 1;
    } else if (d & NO_FEASIBLE_BIT) {
      counters[1] += 1;
    } else if (d < n_variants) {
      count[d] += 1;
      counters[0] += 1;
    } else {
      counters[2] += 1;
    }
  }
  for (uint32_t v = 0; v < n_variants; ++v) {
    const Row &r = rows[v];
    uint64_t drain = (uint64_t)window_us * (uint64_t)r.batch / (uint64_t)r.lat_us;
    if (drain > U32_MAX) drain = U32_MAX;
    uint64_t arrived = (uint64_t)queued[v] + count[v];
    if (arrived > U32_MAX) arrived = U32_MAX;
    queued[v] = (uint32_t)(arrived > drain ? arrived - drain : 0);
    served_total[v] += count[v];
  }
}

}  // extern "C"
