// Measurement aid: sustained rate of plain 32-bit integer lane-operations (add, xor, compare,
// conditional add) over all SMs.  The selection path's second roofline -- the feasibility scan
// counted as 2 compares and 1 AND per list entry examined -- is stated against this number.
#include "common.cuh"

namespace infaas {

namespace {

constexpr int PROBE_THREADS = 1024;
constexpr int PROBE_CHAINS = 8;        // independent dependency chains per thread
constexpr int PROBE_OPS_PER_STEP = 4;  // add, xor, compare, conditional add

__global__ void __launch_bounds__(PROBE_THREADS, 2)
intpipe_probe_kernel(uint32_t iters, uint32_t seed, uint32_t *__restrict__ sink) {
  uint32_t x[PROBE_CHAINS], cnt[PROBE_CHAINS];
  const uint32_t gid = blockIdx.x * blockDim.x + threadIdx.x;
#pragma unroll
  for (int k = 0; k < PROBE_CHAINS; ++k) { x[k] = gid * 2654435761u + k * seed; cnt[k] = 0; }
  const uint32_t c1 = seed | 1u, c2 = seed * 40503u + 7u, y = seed * 97u + 0x40000000u;
  for (uint32_t i = 0; i < iters; ++i) {
#pragma unroll
    for (int k = 0; k < PROBE_CHAINS; ++k) {
      x[k] = (x[k] + c1) ^ c2;          // add, xor
      cnt[k] += x[k] < y;               // compare, conditional add
    }
  }
  uint32_t acc = 0;
#pragma unroll
  for (int k = 0; k < PROBE_CHAINS; ++k) acc += cnt[k] ^ x[k];
  if (acc == 0x9E3779B9u) sink[0] = acc;   // keeps the loop alive; practically never taken
}

}  // namespace

cudaError_t launch_intpipe_probe(uint32_t iters, uint32_t seed, uint32_t *d_sink, int sm_count,
                                 unsigned long long *lane_ops, cudaStream_t stream) {
  const uint32_t grid = (uint32_t)sm_count * 2u;
  intpipe_probe_kernel<<<grid, PROBE_THREADS, 0, stream>>>(iters, seed, d_sink);
  *lane_ops = (unsigned long long)grid * PROBE_THREADS * PROBE_CHAINS * PROBE_OPS_PER_STEP * iters;
  return cudaGetLastError();
}

}  // namespace infaas
