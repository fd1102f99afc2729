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

// Smallest slo that falls in SLO bucket b >= 1 (see common.cuh).
__device__ __forceinline__ uint32_t slo_bucket_floor(uint32_t b) {
  const float f = __uint_as_float((b + SLO_BUCKET_BIAS) << 20);
  return (uint32_t)ceilf(f);     // exact: f < 2^32 and has at most 3 fractional bits
}

// Builds the rank / bitmask index of a list of F <= MASK_MAX_F entries (see common.cuh).
// fr_pred / fr_acc: the list in scan order (shared memory).  Writes into the task block.
__device__ void build_index(unsigned char *block, const BlockLayout &L, uint32_t F,
                            const uint32_t *fr_pred, const uint16_t *fr_acc, uint16_t *rkL,
                            uint16_t *rkA, uint32_t *thr_s, uint16_t *acc_s, uint32_t *meta_out) {
  const uint32_t tid = threadIdx.x, B = blockDim.x;
  // ranks by counting (stable: equal values keep scan order)
  for (uint32_t p = tid; p < F; p += B) {
    const uint32_t pp = fr_pred[p], pa = fr_acc[p];
    uint32_t cl = 0, ca = 0;
    for (uint32_t q = 0; q < F; ++q) {
      const uint32_t qp = fr_pred[q], qa = fr_acc[q];
      cl += (qp < pp) || (qp == pp && q < p);
      ca += (qa < pa) || (qa == pa && q < p);
    }
    rkL[p] = (uint16_t)cl;
    rkA[p] = (uint16_t)ca;
    thr_s[cl] = pp;
    acc_s[ca] = (uint16_t)pa;
  }
  __syncthreads();
  uint32_t *thr_g = reinterpret_cast<uint32_t *>(block + L.thr);
  uint16_t *acc_g = reinterpret_cast<uint16_t *>(block + L.accs);
  for (uint32_t i = tid; i < F; i += B) {
    thr_g[i] = thr_s[i];
    acc_g[i] = acc_s[i];
  }
  // bucket tables
  const uint32_t acc_base = acc_s[0], acc_range = acc_s[F - 1] - acc_s[0];
  uint32_t shift = 0;
  while ((acc_range >> shift) > ACC_BUCKETS - 1) ++shift;
  if (tid == 0) *meta_out = acc_base | (shift << 16);
  unsigned char *startL = block + L.start, *startA = startL + SLO_BUCKET_BYTES;
  for (uint32_t b = tid; b < SLO_BUCKET_BYTES + ACC_BUCKETS; b += B) {
    uint32_t cnt = 0;
    if (b < SLO_BUCKETS) {
      if (b > 0) {
        const uint32_t lo = slo_bucket_floor(b);       // every slo in the bucket is >= lo
        for (uint32_t i = 0; i < F; ++i) cnt += thr_s[i] < lo;
      }
      startL[b] = (unsigned char)min(cnt, 255u);
    } else if (b < SLO_BUCKET_BYTES) {
      startL[b] = 0;
    } else {
      const uint32_t lo = acc_base + ((b - SLO_BUCKET_BYTES) << shift);   // every min_acc in the bucket is >= lo
      for (uint32_t i = 0; i < F; ++i) cnt += acc_s[i] < lo;
      startA[b - SLO_BUCKET_BYTES] = (unsigned char)min(cnt, 255u);
    }
  }
  // masks
  unsigned long long *ML = reinterpret_cast<unsigned long long *>(block + L.masks);
  unsigned long long *MA = ML + (F + 1) * L.nw;
  for (uint32_t idx = tid; idx < (F + 1) * L.nw; idx += B) {
    const uint32_t r = idx / L.nw, w = idx - r * L.nw;
    unsigned long long ml = 0, ma = 0;
    const uint32_t p_end = min(F, 64u * w + 64u);
    for (uint32_t p = 64u * w; p < p_end; ++p) {
      const unsigned long long bit = 1ull << (p & 63u);
      if (rkL[p] < r) ml |= bit;
      if (rkA[p] >= r) ma |= bit;
    }
    ML[idx] = ml;
    MA[idx] = ma;
  }
}

__global__ void rebuild_kernel(DeviceCatalog c, uint32_t sort_n, int advance, uint32_t window_us) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned long long *k64 = reinterpret_cast<unsigned long long *>(smem_raw);   // cost<<32 | pred
  uint32_t *k32 = reinterpret_cast<uint32_t *>(k64 + sort_n);                    // inv_acc<<16 | local
  unsigned char *keep = reinterpret_cast<unsigned char *>(k32 + sort_n);         // 1 = non-dominated
  __shared__ uint32_t warp_sums[32];
  __shared__ uint32_t s_last, s_total;
  __shared__ uint32_t fr_pred[MASK_MAX_F], thr_s[MASK_MAX_F];
  __shared__ uint16_t fr_acc[MASK_MAX_F], rkL[MASK_MAX_F], rkA[MASK_MAX_F], acc_s[MASK_MAX_F];

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

  // 3. prune.  In sorted order every dominator of p sits before p, and every earlier entry
  // q with pred_q <= pred_p and acc_q >= acc_p dominates p (its cost is not larger by the
  // sort, and it differs in some attribute or has the smaller id).
  uint32_t my_kept = 0;
  for (uint32_t p = tid; p < V; p += B) {
    const uint32_t pred_p = (uint32_t)k64[p], inv_p = k32[p] >> 16;
    bool kp = true;
    for (uint32_t q = 0; q < p; ++q) {
      if ((uint32_t)k64[q] <= pred_p && (k32[q] >> 16) <= inv_p) { kp = false; break; }
    }
    keep[p] = kp;
    my_kept += kp;
  }
  if (tid == 0) s_total = 0;
  __syncthreads();
  my_kept = __reduce_add_sync(0xFFFFFFFFu, my_kept);
  if ((tid & 31) == 0 && my_kept) atomicAdd(&s_total, my_kept);
  __syncthreads();
  const uint32_t F = s_total;
  const BlockLayout L = block_layout(F);
  unsigned char *block = c.regions + c.reg_off[t];

  // 4. compact into the task block (scan order)
  unsigned long long *keys_g = reinterpret_cast<unsigned long long *>(block + L.keys);
  uint32_t *ids_g = reinterpret_cast<uint32_t *>(block + L.ids);
  uint32_t kept_so_far = 0;
  for (uint32_t p0 = 0; p0 < V; p0 += B) {      // uniform trip count
    const uint32_t p = p0 + tid;
    const bool kp = p < V && keep[p];
    uint32_t total;
    const uint32_t pos = kept_so_far + block_excl_scan_flag(kp, warp_sums, total);
    if (kp) {
      const uint32_t pred_p = (uint32_t)k64[p], acc = 10000u - (k32[p] >> 16);
      keys_g[pos] = ((unsigned long long)acc << 32) | pred_p;
      ids_g[pos] = c.s_id[base + (k32[p] & 0xFFFFu)];
      if (L.nw) { fr_pred[pos] = pred_p; fr_acc[pos] = (uint16_t)acc; }
    }
    kept_so_far += total;
  }
  __syncthreads();
  if (tid == 0) { c.f_len[t] = F; if (!L.nw) c.f_meta[t] = 0; }
  if (L.nw) build_index(block, L, F, fr_pred, fr_acc, rkL, rkA, thr_s, acc_s, c.f_meta + t);

  // 5. the CTA that finishes last packs all blocks into the image
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
  TaskDesc *desc = reinterpret_cast<TaskDesc *>(c.image);
  const uint32_t desc_bytes = T * (uint32_t)sizeof(TaskDesc);
  // 5a. block offsets = exclusive prefix sum of block sizes (chunks of B tasks, running carry)
  uint32_t carry = desc_bytes, longest = 0, entries = 0, linear = 0;
  __shared__ uint32_t scan_buf[1024];
  bool overflow = false;
  for (uint32_t t0 = 0; t0 < T; t0 += B) {
    const uint32_t tt = t0 + tid;
    const uint32_t len = tt < T ? __ldcg(c.f_len + tt) : 0u;
    const BlockLayout Lt = block_layout(len);
    scan_buf[tid] = Lt.bytes;
    __syncthreads();
    for (uint32_t o = 1; o < B; o <<= 1) {      // Hillis-Steele inclusive scan
      uint32_t v = tid >= o ? scan_buf[tid - o] : 0u;
      __syncthreads();
      scan_buf[tid] += v;
      __syncthreads();
    }
    const uint32_t chunk_total = scan_buf[B - 1];
    const uint32_t incl = scan_buf[tid];
    __syncthreads();                                               // scan_buf is reused below
    if (carry + chunk_total > c.image_capacity) overflow = true;   // uniform
    if (tt < T && !overflow) {
      const uint32_t off = carry + incl - Lt.bytes;
      TaskDesc d;
      d.off_masks = off + Lt.masks;
      d.f_nw = len | (Lt.nw << 16);
      d.acc_meta = __ldcg(c.f_meta + tt);
      d.off_keys = off + Lt.keys;
      d.off_thr = off + Lt.thr;
      d.off_ids = off + Lt.ids;
      d.off_accs = off + Lt.accs;
      d.off_start = off + Lt.start;
      desc[tt] = d;
      // the block's offset, kept for the copy pass
      scan_buf[tid] = off;
    }
    __syncthreads();
    // 5b. copy this chunk's blocks (one warp per task, 16 bytes per lane and step)
    if (!overflow) {
      const uint32_t lane = tid & 31, warp = tid >> 5, nwarps = B >> 5;
      for (uint32_t i = warp; i < B && t0 + i < T; i += nwarps) {
        const uint32_t len_i = __ldcg(c.f_len + t0 + i);
        const uint32_t bytes_i = block_layout(len_i).bytes;
        const uint4 *src = reinterpret_cast<const uint4 *>(c.regions + c.reg_off[t0 + i]);
        uint4 *dst = reinterpret_cast<uint4 *>(c.image + scan_buf[i]);
        for (uint32_t e = lane; e < (bytes_i >> 4); e += 32) dst[e] = __ldcg(src + e);
      }
    }
    longest = max(longest, len);
    entries += len;
    linear += (len > 0 && Lt.nw == 0);
    __syncthreads();
    carry += chunk_total;
  }
  // totals for reporting
  longest = __reduce_max_sync(0xFFFFFFFFu, longest);
  entries = __reduce_add_sync(0xFFFFFFFFu, entries);
  linear = __reduce_add_sync(0xFFFFFFFFu, linear);
  __shared__ uint32_t tot[3];
  if (tid == 0) tot[0] = tot[1] = tot[2] = 0;
  __syncthreads();
  if ((tid & 31) == 0) { atomicMax(&tot[0], longest); atomicAdd(&tot[1], entries); atomicAdd(&tot[2], linear); }
  __syncthreads();
  if (tid == 0) {
    if (overflow) atomicMax(c.err, (uint32_t)DEV_ERR_IMAGE_OVERFLOW);
    c.image_hdr[0] = overflow ? 0xFFFFFFFFu : carry;
    c.image_hdr[1] = tot[0];
    c.image_hdr[2] = tot[1];
    c.image_hdr[3] = tot[2];
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
  uint32_t block = P < 128 ? 128 : (P > 1024 ? 1024 : P);
  size_t smem = (size_t)P * 13;
  rebuild_kernel<<<c.n_tasks, block, smem, stream>>>(c, P, advance_queues ? 1 : 0, window_us);
  return cudaGetLastError();
}

}  // namespace infaas
