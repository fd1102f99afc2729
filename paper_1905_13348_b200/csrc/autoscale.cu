// Scaling-up step of the Model-Autoscaler on the window's tallies (Section 4.2.2, "A Greedy
// Heuristic"; cost function and constraints (1), (2), (4) of Section 4.2.1): one CTA per
// task compares the running variants' saturation throughput with the load they served and,
// if the headroom is too small, prices "replicate the running variant" against "add a faster
// variant of the same architecture".  All arithmetic is unsigned integer arithmetic with
// explicit saturation; the cost is compared as a 128-bit product.
#include "common.cuh"

namespace infaas {
namespace {

constexpr uint32_t AUTOSCALE_THREADS = 256;
constexpr unsigned long long U64_MAX_ = ~0ull;

__device__ __forceinline__ unsigned long long sat_add(unsigned long long a, unsigned long long b) {
  const unsigned long long s = a + b;
  return s < a ? U64_MAX_ : s;
}
__device__ __forceinline__ unsigned long long sat_mul(unsigned long long a, unsigned long long b) {
  return __umul64hi(a, b) ? U64_MAX_ : a * b;
}
// ceil(x * m / 100), saturating at 2^64-1.
__device__ unsigned long long scale_pct_ceil(unsigned long long x, uint32_t m) {
  unsigned long long hi = __umul64hi(x, (unsigned long long)m), lo = x * m;
  const unsigned long long lo99 = lo + 99ull;
  hi += lo99 < lo;
  lo = lo99;
  if (hi >= 100ull) return U64_MAX_;
  // (hi * 2^64 + lo) / 100 by two 64-bit divisions; hi < 100 keeps each quotient below 2^32
  const unsigned long long t1 = (hi << 32) | (lo >> 32);
  const unsigned long long q1 = t1 / 100ull, r1 = t1 % 100ull;
  const unsigned long long t0 = (r1 << 32) | (lo & 0xFFFFFFFFull);
  return (q1 << 32) | (t0 / 100ull);
}

struct Action {            // a candidate, ordered by (cost_hi, cost_lo, kind, id); id ~0 = none
  unsigned long long cost_hi, cost_lo;
  uint32_t kind, id, delta;
};
__device__ __forceinline__ bool better(const Action &a, const Action &b) {
  if (a.id == 0xFFFFFFFFu) return false;
  if (b.id == 0xFFFFFFFFu) return true;
  if (a.cost_hi != b.cost_hi) return a.cost_hi < b.cost_hi;
  if (a.cost_lo != b.cost_lo) return a.cost_lo < b.cost_lo;
  if (a.kind != b.kind) return a.kind < b.kind;
  return a.id < b.id;
}

__global__ void __launch_bounds__(AUTOSCALE_THREADS)
autoscale_kernel(DeviceCatalog c, const uint32_t *s_inst, const uint16_t *s_arch,
                 const unsigned long long *s_qps, const uint32_t *task_slo,
                 uint32_t window_us, uint32_t slack_pct, uint32_t lambda_milli, uint32_t *out_variant,
                 uint32_t *out_delta) {
  __shared__ unsigned long long w_served[AUTOSCALE_THREADS / 32], w_cap[AUTOSCALE_THREADS / 32],
      w_key[AUTOSCALE_THREADS / 32];
  __shared__ uint32_t w_slot[AUTOSCALE_THREADS / 32];
  __shared__ Action w_best[AUTOSCALE_THREADS / 32];
  __shared__ unsigned long long s_deficit;
  __shared__ uint32_t s_r;                       // slot of the running variant, ~0 if none
  const uint32_t t = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t lo = c.task_off[t], hi = c.task_off[t + 1];

  // load served, capacity of what runs, and which running variant served most (ties: lower id)
  unsigned long long served = 0, cap = 0, key = 0;
  uint32_t key_slot = 0xFFFFFFFFu;
  for (uint32_t s = lo + tid; s < hi; s += AUTOSCALE_THREADS) {
    const uint32_t id = c.s_id[s], cnt = c.count_by_id[id], n = s_inst[s];
    served += cnt;
    if (n) {
      cap = sat_add(cap, sat_mul(n, s_qps[s]));
      const unsigned long long k = ((unsigned long long)cnt << 32) | (0xFFFFFFFFu - id);
      if (k > key) { key = k; key_slot = s; }
    }
  }
  for (uint32_t o = 16; o; o >>= 1) {
    served += __shfl_xor_sync(0xFFFFFFFFu, served, o);
    cap = sat_add(cap, __shfl_xor_sync(0xFFFFFFFFu, cap, o));
    const unsigned long long k = __shfl_xor_sync(0xFFFFFFFFu, key, o);
    const uint32_t ks = __shfl_xor_sync(0xFFFFFFFFu, key_slot, o);
    if (k > key) { key = k; key_slot = ks; }
  }
  if (lane == 0) { w_served[warp] = served; w_cap[warp] = cap; w_key[warp] = key; w_slot[warp] = key_slot; }
  __syncthreads();
  if (tid == 0) {
    served = 0; cap = 0; key = 0; key_slot = 0xFFFFFFFFu;
    for (uint32_t w = 0; w < AUTOSCALE_THREADS / 32; ++w) {
      served += w_served[w];
      cap = sat_add(cap, w_cap[w]);
      if (w_key[w] > key) { key = w_key[w]; key_slot = w_slot[w]; }
    }
    if (served > 0xFFFFFFFFull) served = 0xFFFFFFFFull;
    const unsigned long long load = served * 1000000000ull / window_us;
    const unsigned long long need = scale_pct_ceil(load, slack_pct);
    s_deficit = cap >= need ? 0ull : need - cap;
    s_r = key_slot;
  }
  __syncthreads();
  const unsigned long long deficit = s_deficit;
  if (deficit == 0ull) {                          // headroom suffices
    if (tid == 0) { out_variant[t] = INFAAS_AUTOSCALE_NONE; out_delta[t] = 0u; }
    return;
  }
  const uint32_t r = s_r, slo = task_slo[t];
  unsigned long long q_r = 0;
  uint32_t arch_r = 0;
  if (r != 0xFFFFFFFFu) { q_r = s_qps[r]; arch_r = s_arch[r]; }

  Action best;
  best.id = 0xFFFFFFFFu; best.cost_hi = best.cost_lo = 0; best.kind = 0; best.delta = 0;
  for (uint32_t s = lo + tid; s < hi; s += AUTOSCALE_THREADS) {
    const uint32_t lat = c.s_lat[s];
    const unsigned long long q = s_qps[s];               // saturation throughput, milli-queries/s
    if (q == 0ull || lat > slo) continue;         // constraint (2): new instances meet the SLO
    uint32_t kind = 1;                             // 0 replicate, 1 upgrade
    if (s == r) kind = 0;
    else if (r != 0xFFFFFFFFu && (s_arch[s] != arch_r || q <= q_r)) continue;
    const unsigned long long delta = deficit / q + (deficit % q != 0ull);
    if (delta > 0xFFFFFFFFull) continue;
    const unsigned long long a = (unsigned long long)c.s_cost[s] * delta;                 // < 2^64
    const unsigned long long f = 1000000000ull + (unsigned long long)lambda_milli * c.s_load_lat[s];
    Action cand;
    cand.cost_hi = __umul64hi(a, f); cand.cost_lo = a * f;
    cand.kind = kind; cand.id = c.s_id[s]; cand.delta = (uint32_t)delta;
    if (better(cand, best)) best = cand;
  }
  for (uint32_t o = 16; o; o >>= 1) {
    Action other;
    other.cost_hi = __shfl_xor_sync(0xFFFFFFFFu, best.cost_hi, o);
    other.cost_lo = __shfl_xor_sync(0xFFFFFFFFu, best.cost_lo, o);
    other.kind = __shfl_xor_sync(0xFFFFFFFFu, best.kind, o);
    other.id = __shfl_xor_sync(0xFFFFFFFFu, best.id, o);
    other.delta = __shfl_xor_sync(0xFFFFFFFFu, best.delta, o);
    if (better(other, best)) best = other;
  }
  if (lane == 0) w_best[warp] = best;
  __syncthreads();
  if (tid == 0) {
    for (uint32_t w = 1; w < AUTOSCALE_THREADS / 32; ++w)
      if (better(w_best[w], best)) best = w_best[w];
    const bool none = best.id == 0xFFFFFFFFu;
    out_variant[t] = none ? INFAAS_AUTOSCALE_ESCALATE : best.id;
    out_delta[t] = none ? 0u : best.delta;
  }
}

}  // namespace

cudaError_t launch_autoscale(const DeviceCatalog &c, const uint32_t *s_inst, const uint16_t *s_arch,
                             const unsigned long long *s_qps, const uint32_t *task_slo, uint32_t window_us, uint32_t slack_pct,
                             uint32_t lambda_milli, uint32_t *d_variant, uint32_t *d_delta,
                             cudaStream_t stream) {
  autoscale_kernel<<<c.n_tasks, AUTOSCALE_THREADS, 0, stream>>>(c, s_inst, s_arch, s_qps, task_slo, window_us, slack_pct,
                                                                lambda_milli, d_variant, d_delta);
  return cudaGetLastError();
}

}  // namespace infaas
