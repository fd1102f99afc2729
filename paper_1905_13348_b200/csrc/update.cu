// Load tallies, queue recursion, predicted latency and the per-task scan lists.
//
// Section 4.2.2 of the paper tracks the load a variant serves from the queries it is given
// and its batch size; Section 4 says a loaded variant's latency is not its profiled one.
// Here a window's decisions are counted per variant (tally kernel), each variant's queue is
// advanced by one window and its load-adjusted latency recomputed, and every task's list of
// non-dominated variants is rebuilt in (cost, pred_lat, -acc, id) order (rebuild kernel).
#include "common.cuh"

namespace infaas {

namespace {

constexpr uint32_t U32_MAX_ = 0xFFFFFFFFu;

// ------------------------------------------------------------------------------------
// Tally: count[v] += #decisions equal to v.  Lanes of a warp that hold the same variant
// are merged into one atomic (hot variants take most of a hot task's queries).
// ------------------------------------------------------------------------------------
__device__ __forceinline__ void tally_one(uint32_t d, bool live, uint32_t n_variants,
                                          uint32_t *count_by_id, uint32_t &n_feas,
                                          uint32_t &n_nofeas, uint32_t &n_inval) {
  bool feas = live && d < n_variants && !(d & INFAAS_NO_FEASIBLE);
  bool inval = live && !feas && (d == INFAAS_INVALID || !(d & INFAAS_NO_FEASIBLE));
  bool nofeas = live && !feas && !inval;
  n_feas += feas;
  n_nofeas += nofeas;
  n_inval += inval;
  unsigned fm = __ballot_sync(0xFFFFFFFFu, feas);
  if (feas) {
    unsigned peers = __match_any_sync(fm, d);
    int leader = __ffs(peers) - 1;
    if ((threadIdx.x & 31) == leader) atomicAdd(&count_by_id[d], (uint32_t)__popc(peers));
  }
}

__global__ void __launch_bounds__(256)
tally_kernel(const uint32_t *__restrict__ decision, uint64_t n, uint32_t n_variants,
             uint32_t *__restrict__ count_by_id, unsigned long long *__restrict__ counters) {
  __shared__ uint32_t blk[3];
  if (threadIdx.x < 3) blk[threadIdx.x] = 0;
  __syncthreads();
  uint32_t n_feas = 0, n_nofeas = 0, n_inval = 0;
  const uint64_t n4 = n >> 2;
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  const uint4 *dec4 = reinterpret_cast<const uint4 *>(decision);
  // whole warps iterate together so that the warp-wide intrinsics see all 32 lanes
  const uint64_t n4_warp = (n4 + 31) & ~(uint64_t)31;
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4_warp; i += stride) {
    bool live = i < n4;
    uint4 d = live ? __ldg(dec4 + i) : make_uint4(0, 0, 0, 0);
    tally_one(d.x, live, n_variants, count_by_id, n_feas, n_nofeas, n_inval);
    tally_one(d.y, live, n_variants, count_by_id, n_feas, n_nofeas, n_inval);
    tally_one(d.z, live, n_variants, count_by_id, n_feas, n_nofeas, n_inval);
    tally_one(d.w, live, n_variants, count_by_id, n_feas, n_nofeas, n_inval);
  }
  if (blockIdx.x == 0 && threadIdx.x < 32) {  // ragged tail, at most 3 elements
    uint64_t i = (n4 << 2) + threadIdx.x;
    bool live = i < n;
    uint32_t d = live ? decision[i] : 0;
    tally_one(d, live, n_variants, count_by_id, n_feas, n_nofeas, n_inval);
  }
  n_feas = __reduce_add_sync(0xFFFFFFFFu, n_feas);
  n_nofeas = __reduce_add_sync(0xFFFFFFFFu, n_nofeas);
  n_inval = __reduce_add_sync(0xFFFFFFFFu, n_inval);
  if ((threadIdx.x & 31) == 0) {
    atomicAdd(&blk[0], n_feas);
    atomicAdd(&blk[1], n_nofeas);
    atomicAdd(&blk[2], n_inval);
  }
  __syncthreads();
  if (threadIdx.x < 3 && blk[threadIdx.x]) atomicAdd(&counters[threadIdx.x], (unsigned long long)blk[threadIdx.x]);
}

// ------------------------------------------------------------------------------------
// Rebuild: one CTA per task.
// ------------------------------------------------------------------------------------
__device__ __forceinline__ bool key_less(unsigned long long a64, uint32_t a32,
                                         unsigned long long b64, uint32_t b32) {
  return a64 < b64 || (a64 == b64 && a32 < b32);
}

// Exclusive scan of one flag per thread over the CTA; returns this thread's offset and the
// CTA total.  `warp_sums` holds blockDim/32 words.
__device__ __forceinline__ uint32_t block_excl_scan_flag(bool flag, uint32_t *warp_sums,
                                                         uint32_t &total) {
  unsigned b = __ballot_sync(0xFFFFFFFFu, flag);
  uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  uint32_t in_warp = __popc(b & ((1u << lane) - 1u));
  __syncthreads();
  if (lane == 0) warp_sums[warp] = __popc(b);
  __syncthreads();
  uint32_t before = 0, all = 0;
  for (uint32_t w = 0; w < nw; ++w) {
    uint32_t s = warp_sums[w];
    before += (w < warp) ? s : 0;
    all += s;
  }
  total = all;
  return before + in_warp;
}

__global__ void rebuild_kernel(DeviceCatalog c, uint32_t sort_n, int advance, uint32_t window_us) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned long long *k64 = reinterpret_cast<unsigned long long *>(smem_raw);   // cost<<32 | pred
  uint32_t *k32 = reinterpret_cast<uint32_t *>(k64 + sort_n);                    // inv_acc<<16 | local
  __shared__ uint32_t warp_sums[32];
  __shared__ uint32_t s_last;

  const uint32_t t = blockIdx.x, tid = threadIdx.x, B = blockDim.x;
  const uint32_t base = c.task_off[t];
  const uint32_t V = c.task_off[t + 1] - base;

  // sort size for this task: the power of two that holds it (tasks differ in size)
  uint32_t P = 1;
  while (P < V) P <<= 1;

  // 1. queue recursion, predicted latency, sort keys
  for (uint32_t i = tid; i < P; i += B) {
    if (i < V) {
      const uint32_t slot = base + i;
      const uint32_t lat = c.s_lat[slot];
      const uint32_t batch = c.s_batch[slot];
      uint32_t queued = c.s_queued[slot];
      if (advance) {
        const uint32_t id = c.s_id[slot];
        const uint32_t cnt = c.count_by_id[id];
        c.count_by_id[id] = 0;
        c.s_served[slot] += cnt;
        unsigned long long arrived = (unsigned long long)queued + cnt;
        if (arrived > U32_MAX_) arrived = U32_MAX_;
        unsigned long long drain = (unsigned long long)window_us * batch / lat;
        if (drain > U32_MAX_) drain = U32_MAX_;
        queued = arrived > drain ? (uint32_t)(arrived - drain) : 0u;
        c.s_queued[slot] = queued;
      }
      unsigned long long p = (unsigned long long)lat + (unsigned long long)queued * lat / batch;
      const uint32_t pred = p > U32_MAX_ ? U32_MAX_ : (uint32_t)p;
      c.s_pred[slot] = pred;
      k64[i] = ((unsigned long long)c.s_cost[slot] << 32) | pred;
      k32[i] = ((10000u - c.s_acc[slot]) << 16) | i;
    } else {
      k64[i] = ~0ull;
      k32[i] = ~0u;
    }
  }
  __syncthreads();

  // 2. bitonic sort of P keys, ascending in (cost, pred, 10000-acc, local index)
  for (uint32_t k = 2; k <= P; k <<= 1) {
    for (uint32_t j = k >> 1; j > 0; j >>= 1) {
      for (uint32_t x = tid; x < (P >> 1); x += B) {
        uint32_t i = ((x & ~(j - 1)) << 1) | (x & (j - 1));   // lower index of the pair
        uint32_t l = i | j;
        bool up = (i & k) == 0;
        unsigned long long a64 = k64[i], b64 = k64[l];
        uint32_t a32 = k32[i], b32 = k32[l];
        bool swap = up ? key_less(b64, b32, a64, a32) : key_less(a64, a32, b64, b32);
        if (swap) {
          k64[i] = b64; k64[l] = a64;
          k32[i] = b32; k32[l] = a32;
        }
      }
      __syncthreads();
    }
  }

  // 3. prune + 4. compact.  In sorted order every dominator of p sits before p, and every
  // earlier entry q with pred_q <= pred_p and acc_q >= acc_p dominates p (its cost is not
  // larger by the sort, and it differs in some attribute or has the smaller id).
  const uint32_t reg = c.reg_off[t];
  uint32_t kept_so_far = 0;
  for (uint32_t p0 = 0; p0 < V; p0 += B) {      // uniform trip count
    const uint32_t p = p0 + tid;
    bool keep = false;
    uint32_t pred_p = 0, inv_p = 0, local = 0;
    if (p < V) {
      pred_p = (uint32_t)k64[p];
      inv_p = k32[p] >> 16;
      local = k32[p] & 0xFFFFu;
      keep = true;
      for (uint32_t q = 0; q < p; ++q) {
        if ((uint32_t)k64[q] <= pred_p && (k32[q] >> 16) <= inv_p) { keep = false; break; }
      }
    }
    uint32_t total;
    uint32_t off = block_excl_scan_flag(keep, warp_sums, total);
    if (keep) {
      const uint32_t acc = 10000u - inv_p;
      c.f_key[reg + kept_so_far + off] = ((unsigned long long)acc << 32) | pred_p;
      c.f_id[reg + kept_so_far + off] = c.s_id[base + local];
    }
    kept_so_far += total;
  }
  if (tid == 0) c.f_len[t] = kept_so_far;

  // 5. the CTA that finishes last packs all lists into the blob
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    uint32_t ticket = atomicAdd(c.done_ctr, 1u);
    s_last = (ticket == gridDim.x - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();

  const uint32_t T = c.n_tasks;
  uint32_t *table = reinterpret_cast<uint32_t *>(c.blob);
  // 5a. starts = exclusive prefix sum of the lengths (chunks of B tasks, running carry)
  uint32_t carry = 0, longest = 0;
  __shared__ uint32_t scan_buf[1024];
  for (uint32_t t0 = 0; t0 < T; t0 += B) {
    const uint32_t tt = t0 + tid;
    const uint32_t len = tt < T ? __ldcg(c.f_len + tt) : 0u;
    scan_buf[tid] = len;
    __syncthreads();
    for (uint32_t o = 1; o < B; o <<= 1) {      // Hillis-Steele inclusive scan
      uint32_t v = tid >= o ? scan_buf[tid - o] : 0u;
      __syncthreads();
      scan_buf[tid] += v;
      __syncthreads();
    }
    if (tt < T) {
      table[2 * tt] = carry + scan_buf[tid] - len;
      table[2 * tt + 1] = len;
    }
    longest = max(longest, len);
    const uint32_t chunk_total = scan_buf[B - 1];
    __syncthreads();
    carry += chunk_total;
  }
  if (tid == 0 && (T & 1u)) { table[2 * T] = 0; table[2 * T + 1] = 0; }   // pad entry
  const uint32_t E = carry;
  const uint32_t E_pad = (E + 3u) & ~3u;
  const uint32_t bytes = blob_total_bytes(c.n_tasks_pad, E_pad);
  if (bytes > c.blob_capacity) {
    if (tid == 0) { atomicMax(c.err, (uint32_t)DEV_ERR_BLOB_OVERFLOW); *c.done_ctr = 0; }
    return;
  }
  __syncthreads();   // table writes visible to the CTA
  unsigned long long *bkeys = reinterpret_cast<unsigned long long *>(c.blob + blob_table_bytes(c.n_tasks_pad));
  uint32_t *bids = reinterpret_cast<uint32_t *>(bkeys + E_pad);
  // 5b. one warp per task copies its list
  const uint32_t lane = tid & 31, warp = tid >> 5, nw = B >> 5;
  for (uint32_t tt = warp; tt < T; tt += nw) {
    const uint32_t start = table[2 * tt], len = table[2 * tt + 1], r = c.reg_off[tt];
    for (uint32_t e = lane; e < len; e += 32) {
      bkeys[start + e] = __ldcg(c.f_key + r + e);
      bids[start + e] = __ldcg(c.f_id + r + e);
    }
  }
  for (uint32_t e = E + tid; e < E_pad; e += B) {   // padding never matches a query
    bkeys[e] = 0xFFFFFFFFull;                        // pred = 2^32-1, acc = 0
    bids[e] = INFAAS_INVALID;
  }
  // longest list (for reporting)
  longest = __reduce_max_sync(0xFFFFFFFFu, longest);
  if (lane == 0) warp_sums[warp] = longest;
  __syncthreads();
  if (tid == 0) {
    uint32_t m = 0;
    for (uint32_t w = 0; w < nw; ++w) m = max(m, warp_sums[w]);
    c.blob_hdr[0] = bytes;
    c.blob_hdr[1] = E_pad;
    c.blob_hdr[2] = m;
    c.blob_hdr[3] = E;
    *c.done_ctr = 0;
  }
}

}  // namespace

cudaError_t launch_tally(const DeviceCatalog &c, const uint32_t *d_decision, uint64_t n,
                         cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  uint64_t want = ((n >> 2) + 255) / 256;
  uint32_t grid = (uint32_t)(want < 1 ? 1 : (want > 148 * 8 ? 148 * 8 : want));
  tally_kernel<<<grid, 256, 0, stream>>>(d_decision, n, c.n_variants, c.count_by_id, c.counters);
  return cudaGetLastError();
}

cudaError_t prepare_rebuild_kernel() {
  return cudaFuncSetAttribute(rebuild_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)REBUILD_MAX_SMEM);
}

cudaError_t launch_rebuild(const DeviceCatalog &c, bool advance_queues, uint32_t window_us,
                           cudaStream_t stream) {
  uint32_t P = 1;
  while (P < c.max_task_variants) P <<= 1;
  uint32_t block = P < 64 ? 64 : (P > 1024 ? 1024 : P);
  size_t smem = (size_t)P * 12;
  rebuild_kernel<<<c.n_tasks, block, smem, stream>>>(c, P, advance_queues ? 1 : 0, window_us);
  return cudaGetLastError();
}

}  // namespace infaas
