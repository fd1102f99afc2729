// Worker choice for decided queries (Section 4.1, Case I: the query goes to the least-loaded
// worker running an instance of the chosen variant, or, if the variant is not loaded, to the
// least-utilised worker with the variant's hardware; Section 5: an instance is a {variant,
// worker} pair).  All queries of a batch see one snapshot of the two tables, so the answer is
// a function of the variant: a table with one worker per variant is built when the tables are
// given, and the per-query step is a gather through it.
#include "common.cuh"

namespace infaas {
namespace {

constexpr unsigned long long NO_KEY = ~0ull;

__global__ void workers_reset_kernel(unsigned long long *best_inst, uint32_t n_variants,
                                     unsigned long long *best_hw) {
  const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n_variants) best_inst[i] = NO_KEY;
  if (i < 256u) best_hw[i] = NO_KEY;
}

// Smallest (load, worker) per variant over the instance table, smallest (util, worker) per
// hardware code over the worker table.
__global__ void workers_scan_kernel(const uint32_t *inst_variant, const uint32_t *inst_worker,
                                    const uint32_t *inst_load, uint32_t n_inst, uint32_t n_variants,
                                    const unsigned char *worker_hw, const uint32_t *worker_util,
                                    uint32_t n_workers, unsigned long long *best_inst,
                                    unsigned long long *best_hw) {
  const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n_inst) {
    const uint32_t v = inst_variant[i], w = inst_worker[i];
    if (v < n_variants && w < n_workers) atomicMin(best_inst + v, ((unsigned long long)inst_load[i] << 32) | w);
  }
  if (i < n_workers) atomicMin(best_hw + worker_hw[i], ((unsigned long long)worker_util[i] << 32) | i);
}

__global__ void workers_final_kernel(uint32_t n_variants, const unsigned char *hw_by_id,
                                     const unsigned long long *best_inst, const unsigned long long *best_hw,
                                     uint32_t *worker_of) {
  const uint32_t v = blockIdx.x * blockDim.x + threadIdx.x;
  if (v >= n_variants) return;
  unsigned long long k = best_inst[v];
  if (k == NO_KEY) k = best_hw[hw_by_id[v]];
  worker_of[v] = k == NO_KEY ? INFAAS_INVALID : (uint32_t)k;
}

__device__ __forceinline__ uint32_t worker_for(uint32_t d, uint32_t n_variants, const uint32_t *worker_of) {
  return d < n_variants ? __ldg(worker_of + d) : INFAAS_INVALID;     // bit 31 set is >= n_variants too
}

// 8 B per query: four decisions in, four workers out per thread and trip.
__global__ void __launch_bounds__(256)
assign_workers_kernel(const uint32_t *__restrict__ decision, uint64_t n, uint32_t n_variants,
                      const uint32_t *__restrict__ worker_of, uint32_t *__restrict__ worker) {
  const uint64_t n4 = n >> 2, stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
    const uint4 d = __ldcs(reinterpret_cast<const uint4 *>(decision) + i);
    uint4 w;
    w.x = worker_for(d.x, n_variants, worker_of);
    w.y = worker_for(d.y, n_variants, worker_of);
    w.z = worker_for(d.z, n_variants, worker_of);
    w.w = worker_for(d.w, n_variants, worker_of);
    __stcs(reinterpret_cast<uint4 *>(worker) + i, w);
  }
  if (blockIdx.x == 0 && threadIdx.x < (n & 3u)) {
    const uint64_t i = (n4 << 2) + threadIdx.x;
    worker[i] = worker_for(decision[i], n_variants, worker_of);
  }
}

}  // namespace

cudaError_t launch_workers_build(uint32_t n_variants, const unsigned char *hw_by_id,
                                 const uint32_t *inst_variant, const uint32_t *inst_worker,
                                 const uint32_t *inst_load, uint32_t n_inst, const unsigned char *worker_hw,
                                 const uint32_t *worker_util, uint32_t n_workers,
                                 unsigned long long *best_inst, unsigned long long *best_hw,
                                 uint32_t *worker_of, cudaStream_t stream) {
  const uint32_t B = 256;
  const uint32_t m = n_variants > 256u ? n_variants : 256u;
  workers_reset_kernel<<<(m + B - 1) / B, B, 0, stream>>>(best_inst, n_variants, best_hw);
  const uint32_t k = n_inst > n_workers ? n_inst : n_workers;
  if (k)
    workers_scan_kernel<<<(k + B - 1) / B, B, 0, stream>>>(inst_variant, inst_worker, inst_load, n_inst, n_variants,
                                                           worker_hw, worker_util, n_workers, best_inst, best_hw);
  workers_final_kernel<<<(n_variants + B - 1) / B, B, 0, stream>>>(n_variants, hw_by_id, best_inst, best_hw,
                                                                   worker_of);
  return cudaGetLastError();
}

cudaError_t launch_assign_workers(const uint32_t *d_decision, uint64_t n, uint32_t n_variants,
                                  const uint32_t *worker_of, uint32_t *d_worker, int sm_count,
                                  cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  uint64_t want = ((n >> 2) + 255) / 256;
  const uint64_t cap = (uint64_t)sm_count * 8;
  const uint32_t grid = (uint32_t)(want < 1 ? 1 : (want > cap ? cap : want));
  assign_workers_kernel<<<grid, 256, 0, stream>>>(d_decision, n, n_variants, worker_of, d_worker);
  return cudaGetLastError();
}

}  // namespace infaas
