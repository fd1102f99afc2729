// Selection kernel: for each query (task, latency SLO, minimum accuracy) pick the cheapest
// variant of the task that meets both requirements, else flag the nearest miss
// (Section 4.1 of the paper, "Case I: on arrival of a query"; cost objective as in the
// worked example of Section 2.2).
//
// The per-task scan lists are already sorted by (cost, pred_lat, -acc, id) and pruned to
// non-dominated variants, so the answer for a feasible query is the FIRST list entry that
// meets both requirements, and the nearest miss is the first entry with the smallest
// distance.  All lists together are a few tens of KB: each CTA stages the packed image in
// shared memory with bulk asynchronous copies (TMA, mbarrier completion) once and then
// streams queries through it, four per thread per iteration with 128-bit loads and stores.
#include "common.cuh"

namespace infaas {

namespace {

constexpr int SELECT_THREADS = 512;
constexpr uint32_t STAGE_CHUNK = 32768;          // bytes per bulk copy
constexpr uint32_t STAGE_POLL_LIMIT = 1u << 22;  // bounded wait on the staging barrier

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

// Stage `bytes` (multiple of 16) from global `src` (16-byte aligned) into shared `dst`.
// Returns false if the copy did not complete within the poll limit.
__device__ __forceinline__ bool stage_blob(unsigned char *dst, const unsigned char *src,
                                           uint32_t bytes, unsigned long long *mbar) {
  const uint32_t bar = smem_u32(mbar);
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
    for (uint32_t off = 0; off < bytes; off += STAGE_CHUNK) {
      const uint32_t sz = min(STAGE_CHUNK, bytes - off);
      asm volatile(
          "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
          ::"r"(smem_u32(dst + off)), "l"(src + off), "r"(sz), "r"(bar)
          : "memory");
    }
  }
  uint32_t done = 0;
  for (uint32_t it = 0; it < STAGE_POLL_LIMIT && !done; ++it) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar)
        : "memory");
  }
  return __syncthreads_and((int)done) != 0;
}

// One query against its task's list.  table/keys/ids point to shared memory (staged) or to
// the global image.
__device__ __forceinline__ uint32_t decide(const uint2 *__restrict__ table,
                                           const unsigned long long *__restrict__ keys,
                                           const uint32_t *__restrict__ ids, uint32_t n_tasks,
                                           uint32_t task, uint32_t slo, uint32_t min_acc) {
  if (task >= n_tasks) return INFAAS_INVALID;
  const uint2 sl = table[task];
  const uint32_t start = sl.x, len = sl.y;
  if (len == 0) return INFAAS_INVALID;
  const unsigned long long *k = keys + start;
  for (uint32_t i = 0; i < len; ++i) {
    const unsigned long long e = k[i];
    if ((uint32_t)e <= slo && (uint32_t)(e >> 32) >= min_acc) return ids[start + i];
  }
  // nothing meets both: nearest miss, d = 10^4 * over_lat + slo * under_acc (64-bit);
  // strict '<' keeps the first of equal distances, i.e. the smallest (cost, pred, -acc, id)
  unsigned long long best = ~0ull;
  uint32_t best_i = 0;
  for (uint32_t i = 0; i < len; ++i) {
    const unsigned long long e = k[i];
    const uint32_t pred = (uint32_t)e, acc = (uint32_t)(e >> 32);
    const uint32_t over = pred > slo ? pred - slo : 0u;
    const uint32_t under = min_acc > acc ? min_acc - acc : 0u;
    const unsigned long long d = (unsigned long long)over * 10000ull + (unsigned long long)slo * under;
    if (d < best) { best = d; best_i = i; }
  }
  return INFAAS_NO_FEASIBLE | ids[start + best_i];
}

__device__ __forceinline__ void select_body(const unsigned char *image, uint32_t n_tasks,
                                            uint32_t n_tasks_pad, uint32_t e_pad,
                                            const uint16_t *__restrict__ task,
                                            const uint32_t *__restrict__ slo,
                                            const uint16_t *__restrict__ min_acc, uint64_t n,
                                            uint32_t *__restrict__ decision) {
  const uint2 *table = reinterpret_cast<const uint2 *>(image);
  const unsigned long long *keys =
      reinterpret_cast<const unsigned long long *>(image + blob_table_bytes(n_tasks_pad));
  const uint32_t *ids = reinterpret_cast<const uint32_t *>(keys + e_pad);

  const uint64_t n4 = n >> 2;
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  const uint2 *task4 = reinterpret_cast<const uint2 *>(task);
  const uint4 *slo4 = reinterpret_cast<const uint4 *>(slo);
  const uint2 *acc4 = reinterpret_cast<const uint2 *>(min_acc);
  uint4 *dec4 = reinterpret_cast<uint4 *>(decision);
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
    const uint2 t = __ldcs(task4 + i);
    const uint4 s = __ldcs(slo4 + i);
    const uint2 a = __ldcs(acc4 + i);
    uint4 d;
    d.x = decide(table, keys, ids, n_tasks, t.x & 0xFFFFu, s.x, a.x & 0xFFFFu);
    d.y = decide(table, keys, ids, n_tasks, t.x >> 16, s.y, a.x >> 16);
    d.z = decide(table, keys, ids, n_tasks, t.y & 0xFFFFu, s.z, a.y & 0xFFFFu);
    d.w = decide(table, keys, ids, n_tasks, t.y >> 16, s.w, a.y >> 16);
    __stcs(dec4 + i, d);
  }
  if (blockIdx.x == 0 && threadIdx.x < (n & 3)) {   // ragged tail
    const uint64_t q = (n4 << 2) + threadIdx.x;
    decision[q] = decide(table, keys, ids, n_tasks, task[q], slo[q], min_acc[q]);
  }
}

__global__ void __launch_bounds__(SELECT_THREADS)
select_kernel(const unsigned char *__restrict__ blob, const uint32_t *__restrict__ blob_hdr,
              uint32_t n_tasks, uint32_t n_tasks_pad, uint32_t smem_bytes,
              const uint16_t *__restrict__ task, const uint32_t *__restrict__ slo,
              const uint16_t *__restrict__ min_acc, uint64_t n, uint32_t *__restrict__ decision,
              uint32_t *err) {
  extern __shared__ __align__(128) unsigned char image[];
  __shared__ __align__(8) unsigned long long mbar;
  const uint32_t bytes = blob_hdr[0], e_pad = blob_hdr[1];
  if (bytes <= smem_bytes) {
    if (!stage_blob(image, blob, bytes, &mbar)) {
      if (threadIdx.x == 0) atomicMax(err, (uint32_t)DEV_ERR_STAGE_TIMEOUT);
      return;
    }
    select_body(image, n_tasks, n_tasks_pad, e_pad, task, slo, min_acc, n, decision);
  } else {
    // lists do not fit in shared memory: scan them in global memory (L2-resident)
    select_body(blob, n_tasks, n_tasks_pad, e_pad, task, slo, min_acc, n, decision);
  }
}

}  // namespace

cudaError_t prepare_select_kernel() {
  return cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)SELECT_MAX_SMEM);
}

cudaError_t launch_select(const DeviceCatalog &c, const uint16_t *d_task, const uint32_t *d_slo,
                          const uint16_t *d_min_acc, uint64_t n, uint32_t *d_decision,
                          int sm_count, uint32_t smem_bytes, cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  // resident CTAs per SM for this shared-memory size (227 KB usable per SM, 1 KB reserved per CTA)
  uint32_t per_sm = (uint32_t)(233472u / (smem_bytes + 1024u + 64u));
  const uint32_t by_threads = 2048 / SELECT_THREADS;
  if (per_sm > by_threads) per_sm = by_threads;
  if (per_sm < 1) per_sm = 1;
  const uint64_t want = ((n >> 2) + SELECT_THREADS - 1) / SELECT_THREADS;
  uint64_t grid = (uint64_t)sm_count * per_sm;
  if (grid > want) grid = want;
  if (grid < 1) grid = 1;
  select_kernel<<<(uint32_t)grid, SELECT_THREADS, smem_bytes, stream>>>(
      c.blob, c.blob_hdr, c.n_tasks, c.n_tasks_pad, smem_bytes, d_task, d_slo, d_min_acc, n,
      d_decision, c.err);
  return cudaGetLastError();
}

}  // namespace infaas
