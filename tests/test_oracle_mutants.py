"""Do the pins notice a wrong oracle?  Each entry below is a plausible mistake (a swapped key
field, a wrong comparison, a dropped rounding) planted in a scratch copy of the oracle's
source; the pin file named beside it must then fail.  The mistakes live on the CPU, in the
oracle only; nothing here touches the CUDA path."""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

import pytest

ROOT = os.path.abspath(os.path.join(os.path.dirname(__file__), ".."))
SRC = os.path.join(ROOT, "oracle", "infaas_oracle.cpp")

S, F, W, A = ("tests/test_oracle_pins.py", "tests/test_oracle_stateful_pins.py",
              "tests/test_oracle_workers_pins.py", "tests/test_oracle_autoscale_pins.py")

# (name, text in the source, replacement, occurrence (0 = first), pin file that must fail)
MUTANTS = [
    # selection without states
    ("miss key: latency before cost", "Key k{{d, r.cost, p, inv_acc, v}};", "Key k{{d, p, r.cost, inv_acc, v}};", 0, S),
    ("feasible key: latency before cost", "Key k{{0, r.cost, p, inv_acc, v}};", "Key k{{0, p, r.cost, inv_acc, v}};", 0, S),
    ("accuracy must exceed", "(r.acc_bp >= min_acc);", "(r.acc_bp > min_acc);", 0, S),
    ("latency must be below", "bool ok = (p <= slo) &&", "bool ok = (p < slo) &&", 0, S),
    ("distance weight 10^3", "uint64_t d = 10000ull * over_lat", "uint64_t d = 1000ull * over_lat", 0, S),
    ("distance without the slo factor", "+ (uint64_t)slo * under_acc;", "+ 10000ull * under_acc;", 0, S),
    ("lower accuracy preferred", "uint64_t inv_acc = (uint64_t)(10000 - (int)r.acc_bp);", "uint64_t inv_acc = r.acc_bp;", 0, S),
    ("queue in whole batches", "uint64_t wait = (uint64_t)queued * (uint64_t)lat_us / (uint64_t)batch;",
     "uint64_t wait = ((uint64_t)queued + batch - 1) / batch * lat_us;", 0, S),
    ("predicted latency wraps", "return (uint32_t)(p > U32_MAX ? U32_MAX : p);", "return (uint32_t)p;", 0, S),
    ("drain divides first", "uint64_t drain = (uint64_t)window_us * (uint64_t)r.batch / (uint64_t)r.lat_us;",
     "uint64_t drain = (uint64_t)window_us / (uint64_t)r.lat_us * (uint64_t)r.batch;", 0, S),
    ("arrivals wrap", "if (arrived > U32_MAX) arrived = U32_MAX;", "arrived &= U32_MAX;", 0, S),
    ("suggestions are tallied", "} else if (d & NO_FEASIBLE_BIT) {\n      counters[1] += 1;",
     "} else if (d & NO_FEASIBLE_BIT) {\n      counters[1] += 1; if ((d & 0x7FFFFFFFu) < n_variants) count[d & 0x7FFFFFFFu] += 1;", 0, S),
    # state-aware selection
    ("Active miss key: latency before cost", "Key6{{d, 0, r.cost, p, inv_acc, v}}", "Key6{{d, 0, p, r.cost, inv_acc, v}}", 0, F),
    ("Inactive miss key: accuracy before latency", "Key6{{d, 1, e, inv_acc, v, 0}}", "Key6{{d, 1, inv_acc, e, v, 0}}", 0, F),
    ("Inactive match key has the cost", "Key6 k{{e, inv_acc, v, 0, 0, 0}};", "Key6 k{{r.cost, e, inv_acc, v, 0, 0}};", 0, F),
    ("Inactive matches first", "if (have_active) return arg_a;\n  if (have_inactive) return arg_i;",
     "if (have_inactive) return arg_i;\n  if (have_active) return arg_a;", 0, F),
    ("Inactive before Active on equal distance", "Key6{{d, 0, r.cost, p, inv_acc, v}} : Key6{{d, 1,", "Key6{{d, 1, r.cost, p, inv_acc, v}} : Key6{{d, 0,", 0, F),
    ("no loading latency", "uint64_t L = active ? (uint64_t)p : e;", "uint64_t L = p;", 0, F),
    ("combined latency wraps", "if (e > U32_MAX) e = U32_MAX;", "e &= U32_MAX;", 0, F),
    ("Overloaded variants selectable", "if (state[v] != ST_ACTIVE && state[v] != ST_INACTIVE) continue;",
     "if (state[v] == ST_INTERFERED) continue;", 0, F),
    ("activation without queries", "if (state[v] == ST_INACTIVE && count > 0) state[v] = ST_ACTIVE;",
     "if (state[v] == ST_INACTIVE) state[v] = ST_ACTIVE;", 0, F),
    ("overload needs two waiting", "state[v] = queued[v] > 0 ? ST_OVERLOADED : ST_ACTIVE;",
     "state[v] = queued[v] > 1 ? ST_OVERLOADED : ST_ACTIVE;", 0, F),
    # worker choice
    ("equal utilisation: higher worker", "worker_util[w] < best_load) {", "worker_util[w] <= best_load) {", 0, W),
    ("equal load: higher worker", "inst_worker[i] < best_w)) {", "inst_worker[i] > best_w)) {", 0, W),
    ("most-loaded instance", "inst_load[i] < best_load ||", "inst_load[i] > best_load ||", 0, W),
    ("hardware ignored", "if (worker_hw[w] != rows[v].hw) continue;", "", 0, W),
    ("utilisation rule first", "if (!have) {\n      for (uint32_t w = 0;", "have = false; if (!have) {\n      for (uint32_t w = 0;", 0, W),
    # autoscaler step
    ("need rounded down", "((u128)L * slack_pct + 99) / 100;", "((u128)L * slack_pct) / 100;", 0, A),
    ("equal throughput upgrades", "Q(v) <= Q(r)) continue;", "Q(v) < Q(r)) continue;", 0, A),
    ("upgrade first on equal cost", "kind < best_kind)) {", "kind > best_kind)) {", 0, A),
    ("instances rounded down", "u128 delta = (deficit + Q(v) - 1) / Q(v);", "u128 delta = deficit / Q(v);", 0, A),
    ("equal tallies: higher id runs", "count[v] > count[r]) {", "count[v] >= count[r]) {", 0, A),
    ("SLO of new instances ignored", "if (Q(v) == 0 || rows[v].lat_us > task_slo_us[t]) continue;",
     "if (Q(v) == 0) continue;", 0, A),
    ("loading latency free", "(1000000000ull + (uint64_t)lambda_milli * load_lat_us[v]);", "1000000000ull;", 0, A),
]


def _run(tmp, idx):
    name, old, new, occ, pin = MUTANTS[idx]
    text = open(SRC).read()
    pos = -1
    for _ in range(occ + 1):
        pos = text.find(old, pos + 1)
    assert pos >= 0, f"mutant '{name}': its text is no longer in the oracle's source"
    d = os.path.join(tmp, f"m{idx}")
    os.makedirs(d)
    path = os.path.join(d, "infaas_oracle.cpp")
    with open(path, "w") as f:
        f.write(text[:pos] + new + text[pos + len(old):])
    env = dict(os.environ, INFAAS_ORACLE_SRC=path)
    r = subprocess.run([sys.executable, "-m", "pytest", pin, "-x", "-q", "-p", "no:cacheprovider"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    return name, r.returncode, r.stdout[-400:]


def test_every_planted_mistake_fails_a_pin(tmp_path):
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        results = list(ex.map(lambda i: _run(str(tmp_path), i), range(len(MUTANTS))))
    # pytest exits with 1 when tests failed (2+ = it could not run them, e.g. a compile error)
    survived = [(n, rc, out) for n, rc, out in results if rc != 1]
    assert not survived, survived


def test_unchanged_copy_passes(tmp_path):
    """The same machinery on an unmodified copy: the pins pass, so a failure above is the
    mistake's doing."""
    path = os.path.join(str(tmp_path), "infaas_oracle.cpp")
    with open(path, "w") as f:
        f.write(open(SRC).read())
    env = dict(os.environ, INFAAS_ORACLE_SRC=path)
    r = subprocess.run([sys.executable, "-m", "pytest", W, "-x", "-q", "-p", "no:cacheprovider"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-400:]
