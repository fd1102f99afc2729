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

// Same tallies with a private histogram per CTA in shared memory (one u32 bin per variant):
// shared-memory atomics absorb the hot variants, and each CTA adds only its non-zero bins
// to the global counts at the end.  Used when the bins fit and the batch is large.
constexpr int TALLY_SMEM_THREADS = 512;

__global__ void __launch_bounds__(TALLY_SMEM_THREADS)
tally_smem_kernel(const uint32_t *__restrict__ decision, uint64_t n, uint32_t n_variants,
                  uint32_t *__restrict__ count_by_id, unsigned long long *__restrict__ counters) {
  extern __shared__ uint32_t hist[];
  __shared__ uint32_t blk[3];
  for (uint32_t i = threadIdx.x; i < n_variants; i += blockDim.x) hist[i] = 0;
  if (threadIdx.x < 3) blk[threadIdx.x] = 0;
  __syncthreads();
  uint32_t n_feas = 0, n_nofeas = 0, n_inval = 0;
  auto one = [&](uint32_t d) {
    if (d < n_variants) { atomicAdd(&hist[d], 1u); ++n_feas; }   // d < n_variants < 2^31: bit 31 clear
    else if (d != INFAAS_INVALID && (d & INFAAS_NO_FEASIBLE)) ++n_nofeas;
    else ++n_inval;
  };
  const uint64_t n4 = n >> 2;
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  const uint4 *dec4 = reinterpret_cast<const uint4 *>(decision);
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
    const uint4 d = __ldcs(dec4 + i);
    one(d.x); one(d.y); one(d.z); one(d.w);
  }
  if (blockIdx.x == 0 && threadIdx.x < (n & 3)) one(decision[(n4 << 2) + threadIdx.x]);
  n_feas = __reduce_add_sync(0xFFFFFFFFu, n_feas);
  n_nofeas = __reduce_add_sync(0xFFFFFFFFu, n_nofeas);
  n_inval = __reduce_add_sync(0xFFFFFFFFu, n_inval);
  if ((threadIdx.x & 31) == 0) {
    atomicAdd(&blk[0], n_feas);
    atomicAdd(&blk[1], n_nofeas);
    atomicAdd(&blk[2], n_inval);
  }
  __syncthreads();
  for (uint32_t i = threadIdx.x; i < n_variants; i += blockDim.x) {
    const uint32_t h = hist[i];
    if (h) atomicAdd(&count_by_id[i], h);
  }
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

// Top 15 bits of a u32 converted to float toward zero: a monotone, roughly logarithmic
// code (8 exponent bits, 7 mantissa bits).  The selection kernel computes the same code.
__device__ __forceinline__ uint32_t float_code(uint32_t x) {
  return __float_as_uint(__uint2float_rz(x)) >> 16;
}
// Smallest u32 whose float_code is >= code (code > 0).
__device__ __forceinline__ uint32_t float_code_floor(uint32_t code) {
  return __float2uint_ru(__uint_as_float(code << 16));
}

struct IndexScratch {          // shared memory used while building one task's index
  uint32_t pred[256], Pd[256];
  uint16_t acc[256], Ad[256];
  unsigned char idxP[256], idxA[256], firstP[256], firstA[256], order[256];
  uint32_t ks, ka;
};

// Builds the exact index of a list of F <= INDEX_MAX_F entries (layout in common.cuh).
// S.pred / S.acc hold the list in scan order.  Writes the SLO records straight into the
// image, the var block into the task's region, and the task's header words (offsets
// relative to the var block) and var-block size into the per-task arrays.
__device__ void build_index(const DeviceCatalog &c, uint32_t t, uint32_t F, uint32_t V, IndexScratch &S) {
  const uint32_t tid = threadIdx.x, B = blockDim.x;
  unsigned char *region = c.regions + c.reg_off[t];
  // distinct values and their ranks
  for (uint32_t p = tid; p < F; p += B) {
    bool fp = true, fa = true;
    for (uint32_t q = 0; q < p; ++q) {
      fp &= S.pred[q] != S.pred[p];
      fa &= S.acc[q] != S.acc[p];
    }
    S.firstP[p] = fp;
    S.firstA[p] = fa;
  }
  if (tid == 0) { S.ks = 0; S.ka = 0; }
  __syncthreads();
  for (uint32_t p = tid; p < F; p += B) {
    uint32_t rp = 0, ra = 0;
    for (uint32_t q = 0; q < F; ++q) {
      rp += S.firstP[q] && S.pred[q] < S.pred[p];
      ra += S.firstA[q] && S.acc[q] < S.acc[p];
    }
    S.idxP[p] = (unsigned char)rp;
    S.idxA[p] = (unsigned char)ra;
    S.Pd[rp] = S.pred[p];
    S.Ad[ra] = S.acc[p];
    atomicMax(&S.ks, rp + 1);
    atomicMax(&S.ka, ra + 1);
  }
  __syncthreads();
  const uint32_t Ks = S.ks, Ka = S.ka;
  // positions ordered by rank of pred_lat (ties in scan order)
  for (uint32_t p = tid; p < F; p += B) {
    uint32_t o = 0;
    for (uint32_t q = 0; q < F; ++q) o += S.idxP[q] < S.idxP[p] || (S.idxP[q] == S.idxP[p] && q < p);
    S.order[o] = (unsigned char)p;
  }
  __syncthreads();

  // var block layout
  const uint32_t Fp8 = (F + 7u) / 8u;
  const uint32_t acc_min = S.Ad[0] & ~3u;
  const uint32_t nbw = (S.Ad[Ka - 1] - acc_min + 2u + ACC_WORD_BITS - 1u) / ACC_WORD_BITS;
  const uint32_t width = Ka + 1u;
  const uint32_t off_pd = 32u * Fp8, off_bitmap = 64u * Fp8, off_t2 = off_bitmap + 4u * nbw;
  const uint32_t off_aux = (off_t2 + (Ks + 3u) * width + 3u) & ~3u;
  const AuxLayout AL = aux_layout(F, Ks, Ka);
  unsigned char *var = region + region_var_offset(V);
  unsigned char *aux = var + off_aux;

  uint32_t *Pd_hot = reinterpret_cast<uint32_t *>(var + off_pd);
  for (uint32_t i = tid; i < Ks; i += B) Pd_hot[i] = S.Pd[i];
  uint16_t *Ad_hot = reinterpret_cast<uint16_t *>(aux + AL.Ad);
  for (uint32_t i = tid; i < Ka; i += B) Ad_hot[i] = S.Ad[i];
  // what the nearest-miss search reads
  for (uint32_t p = tid; p < F; p += B) {
    aux[AL.order + p] = S.order[p];
    aux[AL.ordRank + p] = S.idxP[S.order[p]];
    aux[AL.idxA + p] = S.idxA[p];
    aux[AL.idxP + p] = S.idxP[p];
  }
  for (uint32_t r = tid; r <= Ks; r += B) {
    uint32_t best = 0xFFu, best_acc = 0, cnt = 0;           // highest accuracy among ranks < r
    for (uint32_t p = 0; p < F; ++p) {
      if (S.idxP[p] < r) {
        ++cnt;
        if (best == 0xFFu || S.acc[p] > best_acc) { best = p; best_acc = S.acc[p]; }
      }
    }
    aux[AL.bestA + r] = (unsigned char)best;
    aux[AL.ordStart + r] = (unsigned char)cnt;
  }
  for (uint32_t k = tid; k <= Ka; k += B) {
    uint32_t best = 0xFFu, best_pred = 0;                    // lowest latency among accuracy ranks >= k
    for (uint32_t p = 0; p < F; ++p) {
      if (S.idxA[p] >= k && (best == 0xFFu || S.pred[p] < best_pred)) { best = p; best_pred = S.pred[p]; }
    }
    aux[AL.bestB + k] = (unsigned char)best;
  }

  // SLO records.  A bucket with two or more values points at row Ks + 1 of T2 (rows Ks + 1
  // and Ks + 2 hold only 0xFF), so such a query goes to the slow path.
  const uint32_t cmin = float_code(S.Pd[0]), cmax = float_code(S.Pd[Ks - 1]);
  uint32_t sh = 0;
  while ((cmax >> sh) - (cmin >> sh) > SLO_BUCKETS - 1) ++sh;
  const uint32_t bmin = cmin >> sh;
  uint32_t *slo_rec = reinterpret_cast<uint32_t *>(c.image + image_slo_offset(c.n_tasks)) + t * SLO_BUCKETS;
  for (uint32_t j = tid; j < SLO_BUCKETS; j += B) {
    uint32_t lb = 0, cnt = 0, thr = 0;
    for (uint32_t i = 0; i < Ks; ++i) {
      const uint32_t b = min(max(float_code(S.Pd[i]) >> sh, bmin) - bmin, SLO_BUCKETS - 1);
      lb += b < j;
      if (b == j) { ++cnt; thr = S.Pd[i]; }
    }
    uint32_t rec = (Ks + 1u) << 24;                           // two or more values: slow path
    if (cnt == 0) {
      rec = lb ? ((lb - 1u) << 24) : 0x00FFFFFFu;             // always one more than lb - 1 (lb = 0 cannot occur)
    } else if (cnt == 1) {
      const uint32_t lo = j ? float_code_floor((bmin + j) << sh) : 0u;
      const uint32_t delta = thr - lo;
      if (delta < 0x01000000u) rec = (lb << 24) | delta;
    }
    slo_rec[j] = rec;
  }

  // accuracy bitmap
  uint32_t *bitmap = reinterpret_cast<uint32_t *>(var + off_bitmap);
  for (uint32_t w = tid; w < nbw; w += B) {
    uint32_t bits = 0, prefix = 0;
    for (uint32_t i = 0; i < Ka; ++i) {
      const uint32_t x = S.Ad[i] - acc_min, xw = x / ACC_WORD_BITS;
      prefix += xw < w;
      if (xw == w) bits |= 1u << (x - xw * ACC_WORD_BITS);
    }
    bitmap[w] = (prefix << 24) | bits;
  }
  // T2, one thread per accuracy rank k: walk the positions in latency-rank order
  unsigned char *T2 = var + off_t2;
  for (uint32_t k = tid; k < width; k += B) {
    uint32_t cur = 0xFFu, o = 0;
    T2[k] = 0xFFu;                                             // r = 0: no latency is met
    for (uint32_t r = 1; r <= Ks; ++r) {
      while (o < F && S.idxP[S.order[o]] == r - 1) {
        const uint32_t p = S.order[o];
        if (S.idxA[p] >= k && p < cur) cur = p;
        ++o;
      }
      T2[r * width + k] = (unsigned char)cur;
    }
    T2[(Ks + 1u) * width + k] = 0xFFu;
    T2[(Ks + 2u) * width + k] = 0xFFu;
  }
  if (tid == 0) {
    c.f_hdr[t] = make_uint4(0u | (acc_min << 18), off_bitmap | (width << 18), off_t2 | (sh << 18),
                            bmin | ((ACC_WORD_BITS * nbw - 1u) << 15));
    c.f_slow[t] = make_uint2(off_aux, F | (Ks << 8) | (Ka << 16));
    c.f_var_bytes[t] = round_up_u32(off_aux + AL.bytes, 64u);
  }
}

__global__ void rebuild_kernel(DeviceCatalog c, uint32_t sort_n, int advance, uint32_t window_us) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned long long *k64 = reinterpret_cast<unsigned long long *>(smem_raw);   // cost<<32 | pred
  uint32_t *k32 = reinterpret_cast<uint32_t *>(k64 + sort_n);                    // inv_acc<<16 | local
  unsigned char *keep = reinterpret_cast<unsigned char *>(k32 + sort_n);         // 1 = non-dominated
  __shared__ uint32_t warp_sums[32];
  __shared__ uint32_t s_last, s_total;
  __shared__ IndexScratch S;

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
    for (uint32_t q0 = 0; q0 < p && kp; q0 += 8) {     // groups of 8, exit between groups
      bool dom = false;
#pragma unroll
      for (uint32_t j = 0; j < 8; ++j) {
        const uint32_t q = min(q0 + j, p - 1);          // clamped repeats are harmless
        dom |= (uint32_t)k64[q] <= pred_p && (k32[q] >> 16) <= inv_p;
      }
      kp = !dom;
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
  const bool indexed = F > 0 && F <= INDEX_MAX_F;
  unsigned char *region = c.regions + c.reg_off[t];

  // 4. compact into the task's region (scan order): keys and ids, and the var block's ids
  unsigned long long *keys_g = reinterpret_cast<unsigned long long *>(region);
  uint32_t *ids_g = reinterpret_cast<uint32_t *>(region + 8u * V);
  uint32_t *var_ids = reinterpret_cast<uint32_t *>(region + region_var_offset(V));
  uint32_t kept_so_far = 0;
  for (uint32_t p0 = 0; p0 < V; p0 += B) {      // uniform trip count
    const uint32_t p = p0 + tid;
    const bool kp = p < V && keep[p];
    uint32_t total;
    const uint32_t pos = kept_so_far + block_excl_scan_flag(kp, warp_sums, total);
    if (kp) {
      const uint32_t pred_p = (uint32_t)k64[p], acc = 10000u - (k32[p] >> 16);
      const uint32_t id = c.s_id[base + (k32[p] & 0xFFFFu)];
      keys_g[pos] = ((unsigned long long)acc << 32) | pred_p;
      ids_g[pos] = id;
      if (indexed) { var_ids[pos] = id; S.pred[pos] = pred_p; S.acc[pos] = (uint16_t)acc; }
    }
    kept_so_far += total;
  }
  __syncthreads();
  if (indexed) {
    build_index(c, t, F, V, S);
  } else if (tid == 0) {
    c.f_var_bytes[t] = 0;
  }
  if (tid == 0) c.f_len[t] = F;

  // 5. the CTA that finishes last packs the var blocks into the image and writes the headers
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
  uint4 *hdr = reinterpret_cast<uint4 *>(c.image);
  uint2 *slow = reinterpret_cast<uint2 *>(c.image + image_slow_offset(T));
  const uint32_t dummy = image_dummy_offset(T), var0 = image_var_offset(T);
  // headers of a task without index: everything points at the dummy block, where the
  // bitmap reads 0 and T2 reads 0xFF ("nothing found")
  const uint4 dummy_hdr = make_uint4(dummy, dummy, dummy + 64u, 0u);
  if (tid < 32) {                               // dummy block, the out-of-range entry and its SLO row
    reinterpret_cast<uint32_t *>(c.image + dummy)[tid] = tid < 16 ? 0u : 0xFFFFFFFFu;
    if (tid == 0) {
      uint4 h = dummy_hdr;
      h.z |= HDR_FLAG_INVALID << 21;
      hdr[T] = h;
      slow[T] = make_uint2(0u, 0u);
    }
  }
  {
    uint32_t *row = reinterpret_cast<uint32_t *>(c.image + image_slo_offset(T)) + T * SLO_BUCKETS;
    for (uint32_t j = tid; j < SLO_BUCKETS; j += B) row[j] = 0u;
  }
  // 5a. var offsets = exclusive prefix sum of the var-block sizes (chunks of B tasks)
  uint32_t carry = 0, longest = 0, entries = 0, not_indexed = 0;
  __shared__ uint32_t scan_buf[1024];
  __shared__ uint32_t s_copy_end;
  bool overflow = var0 > c.image_capacity;
  for (uint32_t t0 = 0; t0 < T; t0 += B) {
    const uint32_t tt = t0 + tid;
    const uint32_t len = tt < T ? __ldcg(c.f_len + tt) : 0u;
    const uint32_t vbytes = tt < T ? __ldcg(c.f_var_bytes + tt) : 0u;
    scan_buf[tid] = vbytes;
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
    if (var0 + carry + chunk_total > c.image_capacity) overflow = true;   // uniform
    const uint32_t off = var0 + carry + incl - vbytes;             // from the start of the image
    // a block that does not end below what the 18-bit offsets can address is left out: the
    // task is then served by the slow path, like one whose list is too long for the index
    const bool addressable = off + vbytes <= IMAGE_OFFSET_LIMIT;
    if (tt < T && !overflow) {
      uint4 h = dummy_hdr;
      uint2 sl = make_uint2(0u, len > 255u ? 0u : len);
      if (len == 0) {
        h.z |= HDR_FLAG_INVALID << 21;
      } else if (vbytes == 0 || !addressable) {
        h.z |= HDR_FLAG_NOT_INDEXED << 21;
        ++not_indexed;
      } else {
        const uint4 rel = __ldcg(c.f_hdr + tt);
        const uint2 srel = __ldcg(c.f_slow + tt);
        h = make_uint4(rel.x + off, rel.y + off, rel.z + off, rel.w);
        sl = make_uint2(srel.x + off, srel.y);
      }
      hdr[tt] = h;
      slow[tt] = sl;
    }
    // offsets stay ascending: empty blocks share the next block's offset, and the blocks
    // that are left out (and the padding past T) form a suffix of sentinels
    scan_buf[tid] = (tt < T && addressable) ? off : 0xFFFFFFFFu;
    if (tid == 0) s_copy_end = var0 + carry;
    __syncthreads();
    if (tt < T && addressable && vbytes) atomicMax(&s_copy_end, off + vbytes);
    __syncthreads();
    // 5b. copy this chunk's var blocks: 16-byte units spread over all threads; a unit finds
    // its block by binary search over the chunk's ascending offsets
    if (!overflow) {
      const uint32_t first = var0 + carry;
      const uint32_t units = (s_copy_end - first) >> 4;
      const uint4 *reg4 = reinterpret_cast<const uint4 *>(c.regions);
      uint4 *img4 = reinterpret_cast<uint4 *>(c.image);
      for (uint32_t u0 = 0; u0 < units; u0 += 4u * B) {
        uint4 v[4];
        uint32_t dst[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t u = u0 + (uint32_t)j * B + tid;
          dst[j] = 0xFFFFFFFFu;
          if (u < units) {
            const uint32_t byte = first + (u << 4);
            uint32_t lo = 0, hi = B;                    // last i with scan_buf[i] <= byte
            while (hi - lo > 1) {
              const uint32_t mid = (lo + hi) >> 1;
              if (scan_buf[mid] <= byte) lo = mid; else hi = mid;
            }
            const uint32_t tsrc = t0 + lo;
            const uint32_t Vt = __ldg(c.task_off + tsrc + 1) - __ldg(c.task_off + tsrc);
            const uint32_t src_byte = __ldg(c.reg_off + tsrc) + region_var_offset(Vt) + (byte - scan_buf[lo]);
            v[j] = __ldcg(reg4 + (src_byte >> 4));
            dst[j] = byte >> 4;
          }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (dst[j] != 0xFFFFFFFFu) img4[dst[j]] = v[j];
      }
    }
    longest = max(longest, len);
    entries += len;
    __syncthreads();
    carry += chunk_total;
  }
  // totals for reporting
  longest = __reduce_max_sync(0xFFFFFFFFu, longest);
  entries = __reduce_add_sync(0xFFFFFFFFu, entries);
  not_indexed = __reduce_add_sync(0xFFFFFFFFu, not_indexed);
  __shared__ uint32_t tot[3];
  if (tid == 0) tot[0] = tot[1] = tot[2] = 0;
  __syncthreads();
  if ((tid & 31) == 0) { atomicMax(&tot[0], longest); atomicAdd(&tot[1], entries); atomicAdd(&tot[2], not_indexed); }
  __syncthreads();
  if (tid == 0) {
    if (overflow) atomicMax(c.err, (uint32_t)DEV_ERR_IMAGE_OVERFLOW);
    c.image_hdr[0] = overflow ? 0xFFFFFFFFu : var0 + carry;
    c.image_hdr[1] = tot[0];
    c.image_hdr[2] = tot[1];
    c.image_hdr[3] = tot[2];
    *c.done_ctr = 0;
  }
}

}  // namespace

constexpr uint32_t TALLY_SMEM_MAX_VARIANTS = 49152;   // 192 KB of bins
constexpr uint64_t TALLY_SMEM_MIN_N = 1u << 18;        // below this the zero/flush passes cost more than they save

cudaError_t launch_tally(const DeviceCatalog &c, const uint32_t *d_decision, uint64_t n,
                         cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  if (n >= TALLY_SMEM_MIN_N && c.n_variants <= TALLY_SMEM_MAX_VARIANTS) {
    const size_t smem = (size_t)c.n_variants * 4;
    const uint32_t per_sm = smem > 100 * 1024 ? 1 : 2;
    uint64_t want = ((n >> 2) + TALLY_SMEM_THREADS * 8 - 1) / (TALLY_SMEM_THREADS * 8);
    uint64_t grid = (uint64_t)148 * per_sm;
    if (grid > want) grid = want;
    if (grid < 1) grid = 1;
    tally_smem_kernel<<<(uint32_t)grid, TALLY_SMEM_THREADS, smem, stream>>>(
        d_decision, n, c.n_variants, c.count_by_id, c.counters);
    return cudaGetLastError();
  }
  uint64_t want = ((n >> 2) + 255) / 256;
  uint32_t grid = (uint32_t)(want < 1 ? 1 : (want > 148 * 8 ? 148 * 8 : want));
  tally_kernel<<<grid, 256, 0, stream>>>(d_decision, n, c.n_variants, c.count_by_id, c.counters);
  return cudaGetLastError();
}

cudaError_t prepare_rebuild_kernel() {
  cudaError_t e = cudaFuncSetAttribute(tally_smem_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)(TALLY_SMEM_MAX_VARIANTS * 4));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(rebuild_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)REBUILD_MAX_SMEM);
}

cudaError_t launch_rebuild(const DeviceCatalog &c, bool advance_queues, uint32_t window_us,
                           cudaStream_t stream) {
  uint32_t P = 1;
  while (P < c.max_task_variants) P <<= 1;
  uint32_t block = P < 256 ? 256 : (P > 1024 ? 1024 : P);
  size_t smem = (size_t)P * 13;
  rebuild_kernel<<<c.n_tasks, block, smem, stream>>>(c, P, advance_queues ? 1 : 0, window_us);
  return cudaGetLastError();
}

}  // namespace infaas
