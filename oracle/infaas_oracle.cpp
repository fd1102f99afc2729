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
//   * Variants have a life cycle (Inactive, Active, Overloaded, Interfered); selection looks
//     at Active variants first, then at Inactive ones with their loading latency added, and
//     avoids Overloaded and Interfered ones (Section 4, state machine; Section 4.1).
//
//   * Each window the Model-Autoscaler compares the running variants' saturation throughput
//     with the load they serve and, when the headroom is too small, picks the cheaper of
//     replicating the running variant and upgrading to a faster one of the same architecture
//     (Section 4.2.1 cost function and constraints; Section 4.2.2 scaling-up algorithm).
//
//   * The query is sent to the least-loaded worker that runs the chosen variant, or, if the
//     variant is not loaded, to the least-utilised worker with its hardware (Section 4.1).
//
// Everything is brute force over the full, unsorted, unpruned catalog.  There is no
// sorting, no pruning, no early exit and no blocking.  Readings of points the paper leaves
// open (ties, the queueing term, the distance used for "closest", the queue recursion, what
// moves a variant between states) are this build's choices; those constants are "parity unpinned" by the paper itself, the
// structure around them is pinned by the tests under tests/ (worked example of Table 2,
// brute-force enumeration, closed forms, exact-rational ordering).
//
// Arithmetic: unsigned integers only.  Latency in microseconds (u32), accuracy in basis
// points (u16), cost in integer units (u32).

#include <algorithm>
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

// ---- state-aware selection (Section 4, "State machine for the lifecycle of model-variants";
// Section 4.1, Case I and "Mitigating performance degradation") ----
// Every variant is in one of four states.  A query is answered in this order:
//   1. Active variants carry no loading latency: among those that meet both requirements,
//      the one with the smallest (cost, pred, 10000-acc, id) -- as in select_one.
//   2. Otherwise Inactive variants, which must be loaded first: with eff = min(2^32-1,
//      pred + load_lat), among those with eff <= slo and acc >= min_acc the one with the
//      lowest combined latency: smallest (eff, 10000-acc, id).
//   3. Otherwise a suggestion (bit 31 set): over the Active and Inactive variants, the one
//      with the smallest distance d = 10000*max(0,L-slo) + slo*max(0,min_acc-acc), L = pred
//      for Active and eff for Inactive; equal distances go to an Active variant before an
//      Inactive one, then by the order of step 1 / step 2.
// Overloaded and Interfered variants are never chosen nor suggested.  A task with no Active
// or Inactive variant answers INVALID.
const uint8_t ST_INACTIVE = 0, ST_ACTIVE = 1, ST_OVERLOADED = 2, ST_INTERFERED = 3;

struct Key6 {
  uint64_t k[6];
};
bool key6_less(const Key6 &a, const Key6 &b) {
  for (int i = 0; i < 6; ++i) {
    if (a.k[i] < b.k[i]) return true;
    if (a.k[i] > b.k[i]) return false;
  }
  return false;
}

uint32_t select_one_stateful(const Row *rows, const uint32_t *queued, const uint8_t *state,
                             const uint32_t *load_lat, const std::vector<uint32_t> &members,
                             uint32_t slo, uint16_t min_acc) {
  bool have_active = false, have_inactive = false, have_any = false;
  Key6 best_a{}, best_i{}, best_m{};
  uint32_t arg_a = 0, arg_i = 0, arg_m = 0;
  for (uint32_t v : members) {
    const Row &r = rows[v];
    if (state[v] != ST_ACTIVE && state[v] != ST_INACTIVE) continue;
    const bool active = state[v] == ST_ACTIVE;
    uint32_t p = pred_lat(r.lat_us, queued[v], r.batch);
    uint64_t e = (uint64_t)p + (uint64_t)load_lat[v];
    if (e > U32_MAX) e = U32_MAX;
    uint64_t L = active ? (uint64_t)p : e;               // latency the query would see
    uint64_t inv_acc = (uint64_t)(10000 - (int)r.acc_bp);
    bool ok = (L <= slo) && (r.acc_bp >= min_acc);
    if (ok && active) {
      Key6 k{{r.cost, p, inv_acc, v, 0, 0}};
      if (!have_active || key6_less(k, best_a)) { best_a = k; arg_a = v; have_active = true; }
    }
    if (ok && !active) {
      Key6 k{{e, inv_acc, v, 0, 0, 0}};
      if (!have_inactive || key6_less(k, best_i)) { best_i = k; arg_i = v; have_inactive = true; }
    }
    uint64_t over_lat = L > slo ? L - slo : 0;
    uint64_t under_acc = min_acc > r.acc_bp ? (uint64_t)(min_acc - r.acc_bp) : 0;
    uint64_t d = 10000ull * over_lat + (uint64_t)slo * under_acc;
    Key6 k = active ? Key6{{d, 0, r.cost, p, inv_acc, v}} : Key6{{d, 1, e, inv_acc, v, 0}};
    if (!have_any || key6_less(k, best_m)) { best_m = k; arg_m = v; have_any = true; }
  }
  if (have_active) return arg_a;
  if (have_inactive) return arg_i;
  if (have_any) return NO_FEASIBLE_BIT | arg_m;
  return INVALID;
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

// State-aware form of oracle_select: `state` and `load_lat_us` hold one entry per variant.
void oracle_select_stateful(const void *rows_v, uint32_t n_variants, uint32_t n_tasks,
                            const uint32_t *queued, const uint8_t *state, const uint32_t *load_lat_us,
                            const uint16_t *task, const uint32_t *slo_us, const uint16_t *min_acc_bp,
                            uint64_t n, uint32_t *decision, int n_threads) {
  const Row *rows = (const Row *)rows_v;
  auto members = members_by_task(rows, n_variants, n_tasks);
  auto work = [&](uint64_t lo, uint64_t hi) {
    for (uint64_t q = lo; q < hi; ++q) {
      if (task[q] >= n_tasks) {
        decision[q] = INVALID;
        continue;
      }
      decision[q] = select_one_stateful(rows, queued, state, load_lat_us, members[task[q]], slo_us[q],
                                        min_acc_bp[q]);
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

// State-aware end of a window: oracle_load_update, then every variant's state follows its
// load (Section 4: a variant is Active once loaded, Overloaded while it serves at its peak
// throughput):
//   Inactive and it was given queries this window          -> Active (it has been loaded)
//   then, Active or Overloaded: queue not empty afterwards -> Overloaded, else Active
//   Interfered stays (it is set from outside, by monitoring).
void oracle_load_update_stateful(const void *rows_v, uint32_t n_variants, uint32_t *queued,
                                 uint64_t *served_total, uint64_t counters[3], uint8_t *state,
                                 const uint32_t *decision, uint64_t n, uint32_t window_us) {
  std::vector<uint64_t> before(served_total, served_total + n_variants);
  oracle_load_update(rows_v, n_variants, queued, served_total, counters, decision, n, window_us);
  for (uint32_t v = 0; v < n_variants; ++v) {
    uint64_t count = served_total[v] - before[v];
    if (state[v] == ST_INACTIVE && count > 0) state[v] = ST_ACTIVE;
    if (state[v] == ST_ACTIVE || state[v] == ST_OVERLOADED)
      state[v] = queued[v] > 0 ? ST_OVERLOADED : ST_ACTIVE;
  }
}

// ---- Model-Autoscaler, scaling-up step (Section 4.2.2, "A Greedy Heuristic", scaling up
// algorithm; cost function and constraints (1), (2), (4) of Section 4.2.1) ----
// Per task (application), from the window's per-variant tallies `count`:
//   Q(v)   = floor(10^9 * batch / lat_us)             saturation throughput, milli-queries/s
//   L      = floor(10^9 * min(2^32-1, sum count) / window_us)   load served, milli-queries/s
//   cap    = sum over running variants (instances > 0) of instances * Q   (saturating, 64 bit)
//   need   = ceil(L * slack_pct / 100)                 (saturating)
//   cap >= need: headroom suffices, no action (variant = 0xFFFFFFFF, delta = 0).
// Otherwise deficit = need - cap, and with r = the running variant that served most queries
// this window (ties: lower id; none if nothing runs), the candidate actions are
//   replicate r:   delta = ceil(deficit / Q(r))
//   upgrade to v:  v != r, same architecture as r and Q(v) > Q(r) (any v with Q(v) > 0 if
//                  nothing runs); delta = ceil(deficit / Q(v)) instances of v are added
// each only if the variant's profiled latency meets the task's SLO (constraint (2)) and delta
// fits 32 bits.  The action with the smallest  cost * delta * (10^9 + lambda_milli * load_lat_us)
// wins -- the paper's C (delta + lambda T_load delta) in units of 10^-9 -- replication first on
// equal cost, then the lower id.  No candidate: variant = 0xFFFFFFFE (the step to the
// VM-level autoscaler), delta = 0.
const uint32_t AUTOSCALE_NONE = 0xFFFFFFFFu, AUTOSCALE_ESCALATE = 0xFFFFFFFEu;
typedef unsigned __int128 u128;
const uint64_t U64_MAX = ~0ull;

void oracle_autoscale_step(const void *rows_v, uint32_t n_variants, uint32_t n_tasks,
                           const uint32_t *count, const uint32_t *instances,
                           const uint32_t *load_lat_us, const uint32_t *task_slo_us,
                           uint32_t window_us, uint32_t slack_pct, uint32_t lambda_milli,
                           uint32_t *action_variant, uint32_t *action_delta) {
  const Row *rows = (const Row *)rows_v;
  auto members = members_by_task(rows, n_variants, n_tasks);
  auto Q = [&](uint32_t v) { return (uint64_t)(1000000000ull * rows[v].batch / rows[v].lat_us); };
  for (uint32_t t = 0; t < n_tasks; ++t) {
    action_variant[t] = AUTOSCALE_NONE;
    action_delta[t] = 0;
    u128 served = 0, cap = 0;
    bool have_r = false;
    uint32_t r = 0;
    for (uint32_t v : members[t]) {
      served += count[v];
      if (instances[v] == 0) continue;
      cap += (u128)instances[v] * Q(v);
      if (!have_r || count[v] > count[r]) { r = v; have_r = true; }   // ascending id: ties keep the lower
    }
    if (served > U32_MAX) served = U32_MAX;
    if (cap > U64_MAX) cap = U64_MAX;
    uint64_t L = (uint64_t)(served * 1000000000ull / window_us);
    u128 need = ((u128)L * slack_pct + 99) / 100;
    if (need > U64_MAX) need = U64_MAX;
    if (cap >= need) continue;
    u128 deficit = need - cap;
    bool have_best = false;
    u128 best_cost = 0;
    uint32_t best_kind = 0, best_v = 0, best_delta = 0;
    for (uint32_t v : members[t]) {
      uint32_t kind;                                        // 0 replicate, 1 upgrade
      if (have_r && v == r) kind = 0;
      else if (have_r) {
        if (rows[v].arch != rows[r].arch || Q(v) <= Q(r)) continue;
        kind = 1;
      } else kind = 1;
      if (Q(v) == 0 || rows[v].lat_us > task_slo_us[t]) continue;
      u128 delta = (deficit + Q(v) - 1) / Q(v);
      if (delta > U32_MAX) continue;
      u128 cost = (u128)rows[v].cost * delta * (1000000000ull + (uint64_t)lambda_milli * load_lat_us[v]);
      if (!have_best || cost < best_cost || (cost == best_cost && kind < best_kind)) {
        have_best = true; best_cost = cost; best_kind = kind; best_v = v; best_delta = (uint32_t)delta;
      }
    }
    action_variant[t] = have_best ? best_v : AUTOSCALE_ESCALATE;
    action_delta[t] = have_best ? best_delta : 0;
  }
}

// ---- worker choice (Section 4.1, Case I: the Active variant's query goes to the least-loaded
// worker running an instance of it, an Inactive variant's to the worker with the lowest
// utilisation on the variant's target hardware; Section 5: an instance is a {variant, worker}
// pair) ----
// Per query with a feasible decision v (bit 31 clear, v < n_variants), against one snapshot:
//   some instance of v exists: the worker of the instance with the smallest (load, worker);
//   else: the worker with the smallest (util, worker index) among workers whose hardware code
//   equals hw(v); none: 0xFFFFFFFF.  Other decisions: 0xFFFFFFFF.
void oracle_assign_workers(const void *rows_v, uint32_t n_variants, const uint32_t *inst_variant,
                           const uint32_t *inst_worker, const uint32_t *inst_load, uint32_t n_inst,
                           const uint8_t *worker_hw, const uint32_t *worker_util, uint32_t n_workers,
                           const uint32_t *decision, uint64_t n, uint32_t *worker) {
  const Row *rows = (const Row *)rows_v;
  for (uint64_t q = 0; q < n; ++q) {
    uint32_t v = decision[q];
    worker[q] = INVALID;
    if ((v & NO_FEASIBLE_BIT) || v >= n_variants) continue;
    bool have = false;
    uint64_t best_load = 0, best_w = 0;
    for (uint32_t i = 0; i < n_inst; ++i) {
      if (inst_variant[i] != v || inst_worker[i] >= n_workers) continue;
      if (!have || inst_load[i] < best_load || (inst_load[i] == best_load && inst_worker[i] < best_w)) {
        have = true; best_load = inst_load[i]; best_w = inst_worker[i];
      }
    }
    if (!have) {
      for (uint32_t w = 0; w < n_workers; ++w) {
        if (worker_hw[w] != rows[v].hw) continue;
        if (!have || worker_util[w] < best_load) { have = true; best_load = worker_util[w]; best_w = w; }
      }
    }
    if (have) worker[q] = (uint32_t)best_w;
  }
}

// ---- scan-operation count (a measurement aid for the benchmark, not part of the method) ----
// The cheapest feasible variant can be found by scanning, in (cost, pred, 10000-acc, id) order,
// only the variants of the task that no other variant of it dominates -- B is dominated by A when
// pred(A) <= pred(B), acc(A) >= acc(B), cost(A) <= cost(B) and one of the three is strict or
// id(A) < id(B): whenever B is feasible so is A, and A sorts first.  oracle_frontier writes that
// list for one task.  oracle_scan_ops charges every query the integer operations such a scan
// needs, 32 entries at a time:
//   feasible decision found at 1-based position pos:  3 * 32 * ceil(pos / 32)   (2 compares and
//       1 AND per entry looked at)
//   nothing feasible:  3 * F + 6 * F   (the whole list once for feasibility, once for the 64-bit
//       distance, counted as 6 operations per entry)
//   invalid query: 0
// pos_out (may be NULL) receives each query's 0-based list position, 0xFFFFFFFF where there is none.
static std::vector<uint32_t> frontier_of(const Row *rows, const uint32_t *queued,
                                         const std::vector<uint32_t> &members) {
  std::vector<uint32_t> keep;
  for (uint32_t b : members) {
    const uint32_t pb = pred_lat(rows[b].lat_us, queued[b], rows[b].batch);
    bool dominated = false;
    for (uint32_t a : members) {
      if (a == b) continue;
      const uint32_t pa = pred_lat(rows[a].lat_us, queued[a], rows[a].batch);
      if (pa <= pb && rows[a].acc_bp >= rows[b].acc_bp && rows[a].cost <= rows[b].cost &&
          (pa < pb || rows[a].acc_bp > rows[b].acc_bp || rows[a].cost < rows[b].cost || a < b)) {
        dominated = true;
        break;
      }
    }
    if (!dominated) keep.push_back(b);
  }
  std::sort(keep.begin(), keep.end(), [&](uint32_t x, uint32_t y) {
    Key kx{{0, rows[x].cost, pred_lat(rows[x].lat_us, queued[x], rows[x].batch), (uint64_t)(10000 - (int)rows[x].acc_bp), x}};
    Key ky{{0, rows[y].cost, pred_lat(rows[y].lat_us, queued[y], rows[y].batch), (uint64_t)(10000 - (int)rows[y].acc_bp), y}};
    return key_less(kx, ky);
  });
  return keep;
}

uint32_t oracle_frontier(const void *rows_v, uint32_t n_variants, uint32_t n_tasks, const uint32_t *queued,
                         uint32_t task, uint32_t *ids_out, uint32_t cap) {
  const Row *rows = (const Row *)rows_v;
  auto members = members_by_task(rows, n_variants, n_tasks);
  if (task >= n_tasks) return 0;
  auto f = frontier_of(rows, queued, members[task]);
  for (uint32_t i = 0; i < f.size() && i < cap; ++i) ids_out[i] = f[i];
  return (uint32_t)f.size();
}

uint64_t oracle_scan_ops(const void *rows_v, uint32_t n_variants, uint32_t n_tasks, const uint32_t *queued,
                         const uint16_t *task, const uint32_t *decision, uint64_t n, uint32_t *pos_out) {
  const Row *rows = (const Row *)rows_v;
  auto members = members_by_task(rows, n_variants, n_tasks);
  std::vector<std::vector<uint32_t>> lists(n_tasks);
  std::vector<uint32_t> pos_of(n_variants, 0xFFFFFFFFu);
  for (uint32_t t = 0; t < n_tasks; ++t) {
    lists[t] = frontier_of(rows, queued, members[t]);
    for (uint32_t i = 0; i < lists[t].size(); ++i) pos_of[lists[t][i]] = i;
  }
  uint64_t ops = 0;
  for (uint64_t q = 0; q < n; ++q) {
    const uint32_t d = decision[q];
    uint32_t pos = 0xFFFFFFFFu;
    if (d != INVALID && task[q] < n_tasks) {
      const uint64_t F = lists[task[q]].size();
      if (d & NO_FEASIBLE_BIT) ops += 9 * F;
      else if (d < n_variants && pos_of[d] != 0xFFFFFFFFu) {
        pos = pos_of[d];
        ops += 3ull * 32ull * ((uint64_t)pos / 32 + 1);
      }
    }
    if (pos_out) pos_out[q] = pos;
  }
  return ops;
}

}  // extern "C"
