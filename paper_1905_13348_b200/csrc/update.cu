// Load tallies, queue recursion, predicted latency and the per-task scan lists.
//
// Section 4.2.2 of the paper tracks the load a variant serves from the queries it is given
// and its batch size; Section 4 says a loaded variant's latency is not its profiled one.
// Here a window's decisions are counted per variant (tally kernel), each variant's queue is
// advanced by one window and its load-adjusted latency recomputed, and every task's list of
// non-dominated variants is rebuilt in (cost, pred_lat, -acc, id) order (rebuild kernel).
// On a state-aware catalog the same step moves the variants' life-cycle states with the load
// (Section 4, state machine) and builds the Active and the Inactive list of every task.
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
// to the global counts at the end.  Used when the batch is large.  If the bins of all
// variants do not fit, the ids are split into `parts` ranges of `bins` ids: CTA b counts
// range b % parts over the share b / parts of the decisions (every range sees all
// decisions); the counters come from range 0 alone.
constexpr int TALLY_SMEM_THREADS = 1024;

__global__ void __launch_bounds__(TALLY_SMEM_THREADS)
tally_smem_kernel(const uint32_t *__restrict__ decision, uint64_t n, uint32_t n_variants, uint32_t bins,
                  uint32_t parts, uint32_t *__restrict__ count_by_id,
                  unsigned long long *__restrict__ counters) {
  extern __shared__ uint32_t hist[];
  __shared__ uint32_t blk[3];
  const uint32_t part = blockIdx.x % parts, lo = part * bins, share = blockIdx.x / parts;
  const uint32_t my_bins = min(bins, n_variants - lo);
  const uint32_t spare = my_bins + (threadIdx.x & 31u);
  for (uint32_t i = threadIdx.x; i < my_bins; i += blockDim.x) hist[i] = 0;
  if (threadIdx.x < 3) blk[threadIdx.x] = 0;
  __syncthreads();
  // per decision: one shared-memory atomic and two counters; invalid
  // decisions are what remains of the total
  uint32_t n_feas = 0, n_nofeas = 0, n_seen = 0;
  auto one = [&](uint32_t d) {
    // no branch: what is not in this CTA's range (ids below lo wrap around) lands in one of 32
    // spare bins, one per lane, that nobody reads
    atomicAdd(&hist[min(d - lo, spare)], 1u);
    n_feas += d < n_variants;                                    // d < n_variants < 2^31: bit 31 clear
    n_nofeas += (d - INFAAS_NO_FEASIBLE) < 0x7FFFFFFFu;          // bit 31 set and not INFAAS_INVALID
  };
  const uint32_t n4 = (uint32_t)(n >> 2);                        // n <= 2^32 - 1 (checked by the caller)
  const uint32_t stride = (gridDim.x / parts) * blockDim.x;
  const uint4 *dec4 = reinterpret_cast<const uint4 *>(decision);
  // four 128-bit loads in flight per thread
  uint32_t i = share * blockDim.x + threadIdx.x;
  for (; n4 >= 3 * stride && i < n4 - 3 * stride; i += 4 * stride) {
    const uint4 d0 = __ldcs(dec4 + i), d1 = __ldcs(dec4 + i + stride);
    const uint4 d2 = __ldcs(dec4 + i + 2 * stride), d3 = __ldcs(dec4 + i + 3 * stride);
    one(d0.x); one(d0.y); one(d0.z); one(d0.w);
    one(d1.x); one(d1.y); one(d1.z); one(d1.w);
    one(d2.x); one(d2.y); one(d2.z); one(d2.w);
    one(d3.x); one(d3.y); one(d3.z); one(d3.w);
    n_seen += 16;
  }
  for (; i < n4; i += stride) {
    const uint4 d = __ldcs(dec4 + i);
    one(d.x); one(d.y); one(d.z); one(d.w);
    n_seen += 4;
  }
  if (share == 0 && threadIdx.x < (n & 3)) { one(decision[((uint64_t)n4 << 2) + threadIdx.x]); ++n_seen; }
  uint32_t n_inval = n_seen - n_feas - n_nofeas;
  n_feas = __reduce_add_sync(0xFFFFFFFFu, n_feas);
  n_nofeas = __reduce_add_sync(0xFFFFFFFFu, n_nofeas);
  n_inval = __reduce_add_sync(0xFFFFFFFFu, n_inval);
  if ((threadIdx.x & 31) == 0 && part == 0) {
    atomicAdd(&blk[0], n_feas);
    atomicAdd(&blk[1], n_nofeas);
    atomicAdd(&blk[2], n_inval);
  }
  __syncthreads();
  for (uint32_t i = threadIdx.x; i < my_bins; i += blockDim.x) {
    const uint32_t h = hist[i];
    if (h) atomicAdd(&count_by_id[lo + i], h);
  }
  if (threadIdx.x < 3 && blk[threadIdx.x]) atomicAdd(&counters[threadIdx.x], (unsigned long long)blk[threadIdx.x]);
}

// ------------------------------------------------------------------------------------
// Rebuild: one CTA per task.
// ------------------------------------------------------------------------------------
__device__ __forceinline__ bool key_less(unsigned long long a64, uint32_t a32,
                                         unsigned long long b64, uint32_t b32) {
  return (a64 < b64) | ((a64 == b64) & (a32 < b32));
}
// Packed attributes (cost, pred, 10000 - acc, local index): does b dominate a?  Not worse in
// any of the three, and different in one of them or with the smaller index.  Branch-free.
__device__ __forceinline__ uint32_t dominates(const uint4 b, const uint4 a) {
  return (uint32_t)((b.x <= a.x) & (b.y <= a.y) & (b.z <= a.z) &
                    ((b.x != a.x) | (b.y != a.y) | (b.z != a.z) | (b.w < a.w)));
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

// IEEE-754 pattern of a u32 converted to float toward zero: a monotone, roughly logarithmic
// code.  The selection kernel derives the same bucket from it.
__device__ __forceinline__ uint32_t float_bits(uint32_t x) { return __float_as_uint(__uint2float_rz(x)); }
// Smallest u32 whose float_bits is >= pattern (pattern below that of 2^32).
__device__ __forceinline__ uint32_t float_bits_floor(uint32_t pattern) {
  return __float2uint_ru(__uint_as_float(pattern));
}
constexpr uint32_t BITS_OF_2_POW_32 = 0x4F800000u;

struct IndexScratch {          // shared memory used while building one task's index
  uint32_t pred[256], Pd[256], ids[256];
  uint16_t acc[256], Ad[256];
  unsigned char idxP[256], idxA[256], firstP[256], firstA[256], on_stair[256];
  uint32_t bcnt[256], bthr[256];    // per SLO bucket: distinct latencies inside it, one of them
  uint32_t wbits[MAX_ACC_WORDS];    // per bitmap word: the accuracies present
  unsigned long long Lmask[4][256], Amask[4][256];   // [word][rank]: positions by latency rank < r / accuracy rank >= k
  // per latency rank: the most accurate entry (acc << 16 | 0xFFFF - position, 0 = none) and
  // 1 + position of its stair entry (0 = none); per accuracy rank: the fastest entry
  // (pred << 32 | position, ~0 = none); then their running maximum / minimum / count
  uint32_t rankA[256];
  unsigned long long rankB[256];
  uint16_t stair_at[256];
  uint32_t bestA[257];
  unsigned long long bestB[257];
  unsigned char ord_start[257];
  uint32_t ks, ka, base, fs;
};

// Scans over at most 257 per-rank values by one warp, 32 at a time with a carry.
// out[r] = max of in[0 .. r-1] (0 for r = 0), r = 0 .. n.
__device__ __forceinline__ void warp_prefix_max(const uint32_t *in, uint32_t *out, uint32_t n) {
  const uint32_t lane = threadIdx.x & 31u;
  uint32_t carry = 0;
  for (uint32_t c0 = 0; c0 <= n; c0 += 32) {
    const uint32_t i = c0 + lane;
    uint32_t x = i < n ? in[i] : 0u;
#pragma unroll
    for (uint32_t o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, x, o);
      if (lane >= o) x = max(x, y);
    }
    uint32_t before = __shfl_up_sync(0xFFFFFFFFu, x, 1);
    before = max(lane ? before : 0u, carry);
    if (i <= n) out[i] = before;
    carry = max(carry, __shfl_sync(0xFFFFFFFFu, x, 31));
  }
}
// out[k] = min of in[k .. n-1] (~0 for k = n), k = 0 .. n.
__device__ __forceinline__ void warp_suffix_min(const unsigned long long *in, unsigned long long *out, uint32_t n) {
  const uint32_t lane = threadIdx.x & 31u;
  unsigned long long carry = ~0ull;
  if (lane == 0) out[n] = ~0ull;
  for (uint32_t c0 = 0; c0 < n; c0 += 32) {              // from the top down
    const uint32_t q = c0 + lane;                          // q-th element from the top
    unsigned long long x = q < n ? in[n - 1u - q] : ~0ull;
#pragma unroll
    for (uint32_t o = 1; o < 32; o <<= 1) {
      const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, x, o);
      if (lane >= o) x = min(x, y);
    }
    if (q < n) out[n - 1u - q] = min(x, carry);
    carry = min(carry, __shfl_sync(0xFFFFFFFFu, x, 31));
  }
}
// out[r] = number of non-zero in[0 .. r-1], r = 0 .. n.
__device__ __forceinline__ void warp_prefix_count(const uint16_t *in, unsigned char *out, uint32_t n) {
  const uint32_t lane = threadIdx.x & 31u;
  uint32_t carry = 0;
  for (uint32_t c0 = 0; c0 <= n; c0 += 32) {
    const uint32_t i = c0 + lane;
    const unsigned m = __ballot_sync(0xFFFFFFFFu, i < n && in[i] != 0);
    if (i <= n) out[i] = (unsigned char)(carry + __popc(m & ((1u << lane) - 1u)));
    carry += __popc(m);
  }
}

// Fixed part of the image for a task without index (also entry n_tasks): a header word,
// records and a bitmap that make every query of the task read "none".  All threads.
__device__ __forceinline__ void write_dummy_task(const DeviceCatalog &c, uint32_t t) {
  const uint32_t T = c.n_tasks;
  if (threadIdx.x == 0) reinterpret_cast<uint32_t *>(c.image + IMAGE_HDR_OFFSET)[t] = DUMMY_HEADER;
  uint32_t *rec = reinterpret_cast<uint32_t *>(c.image + image_rec_offset(T) + t * REC_STRIDE);
  for (uint32_t j = threadIdx.x; j < SLO_BUCKETS; j += blockDim.x) rec[j] = 0u;
  uint32_t *bm = reinterpret_cast<uint32_t *>(c.image + image_bitmap_offset(T) + t * bitmap_stride(c.nbw));
  for (uint32_t j = threadIdx.x; j < c.nbw; j += blockDim.x) bm[j] = 0u;
}

// Bucket scale of the SLO records: S (16..23) and bmin such that SLO_BUCKETS - 1 buckets of
// 2^S float patterns cover everything from the catalog's smallest profiled latency up to the
// largest SLO asked for so far (as a bit mask: every SLO seen is <= cap).
__device__ __forceinline__ void bucket_scale(const DeviceCatalog &c, uint32_t &Sh, uint32_t &bmin) {
  uint32_t cap = *c.slo_seen | SLO_CAP_FLOOR_US;
  cap |= cap >> 1; cap |= cap >> 2; cap |= cap >> 4; cap |= cap >> 8; cap |= cap >> 16;
  const uint32_t clo = c.lat_code_lo;
  const uint32_t chi = max(clo, __float_as_uint(__uint2float_rz(cap)) >> 16);
  uint32_t sh = 0;
  while ((chi >> sh) - (clo >> sh) > SLO_BUCKETS - 2) ++sh;
  bmin = clo >> sh;
  Sh = 16u + sh;
}

// Sum / OR over the aligned group of 8 lanes this lane belongs to.
__device__ __forceinline__ uint32_t group8_add(uint32_t v) {
  v += __shfl_xor_sync(0xFFFFFFFFu, v, 1);
  v += __shfl_xor_sync(0xFFFFFFFFu, v, 2);
  v += __shfl_xor_sync(0xFFFFFFFFu, v, 4);
  return v;
}
__device__ __forceinline__ uint32_t group8_or(uint32_t v) {
  v |= __shfl_xor_sync(0xFFFFFFFFu, v, 1);
  v |= __shfl_xor_sync(0xFFFFFFFFu, v, 2);
  v |= __shfl_xor_sync(0xFFFFFFFFu, v, 4);
  return v;
}

// One atomic per allocation places a block in the image and, on a CTA's last allocation
// (`done`), counts the CTA as finished with the cursor.  The CTA that is counted last knows the
// final image size: it publishes it for the kernels that follow and clears the counter for the
// next rebuild.  Thread 0 only, in two halves so that the atomic's round trip can overlap other
// work: place_block_issue returns the counter's old value, place_block_finish (same arguments)
// the block's offset behind the fixed part of the image.
__device__ __forceinline__ unsigned long long place_block_issue(const DeviceCatalog &c, uint32_t bytes, bool done) {
  return atomicAdd(c.alloc_ctr, ((unsigned long long)(done ? 1u : 0u) << 32) | bytes);
}
__device__ __forceinline__ uint32_t place_block_finish(const DeviceCatalog &c, unsigned long long old,
                                                       uint32_t bytes, bool done) {
  if (done && (uint32_t)(old >> 32) == gridDim.x - 1u) {
    c.image_hdr[0] = image_var_offset(c.n_tasks, c.nbw) + (uint32_t)old + bytes;
    *c.alloc_ctr = 0ull;
  }
  return (uint32_t)old;
}

// Builds the exact index of a list of F <= INDEX_MAX_F entries (layout in common.cuh) into
// a block of the image obtained from the block cursor.  S.pred / S.acc / S.ids hold the
// list in scan order.  Returns false (all threads) if the list cannot be indexed: its block
// lies beyond the image's capacity or beyond what the header's offset field addresses.  blockDim = REBUILD_THREADS: the pair loops give every entry 8 lanes, and
// the tables, which do not depend on each other, are written by different groups of warps.
// `xi`: 0xFFFFFFFF for the task's first segment (header word, SLO records and bitmap go into the
// fixed part of the image), else the index of this further segment (header to xhdr[xi], bitmap
// into the block, no records: only the slow path comes here).  `next`: 1 + index of the task's next segment, 0 if this is the last (the CTA's last
// allocation, then).
__device__ bool build_index(const DeviceCatalog &c, uint32_t t, uint32_t F, IndexScratch &S, uint32_t xi,
                            uint32_t next) {
  const uint32_t tid = threadIdx.x, B = blockDim.x;
  const bool first = xi == 0xFFFFFFFFu;
  const uint32_t sub = tid & 7u, PB = B >> 3;          // lane of the entry's group; entries per pass
  // distinct values ...
  for (uint32_t p0 = 0; p0 < F; p0 += PB) {            // uniform trip count
    const uint32_t p = p0 + (tid >> 3);
    // bit 0: an earlier entry has this latency; bit 1: this accuracy; bit 2: some entry is at
    // least as fast and at least as accurate, and better in one of the two or, being equal in
    // both (an Active and an Inactive entry can be), earlier
    uint32_t dup = 0;
    if (p < F) {
      const uint32_t pp = S.pred[p], pa = S.acc[p];
#pragma unroll 4
      for (uint32_t q = sub; q < F; q += 8) {              // no branches: the trips' loads overlap
        const uint32_t qp = S.pred[q], qa = S.acc[q];
        const uint32_t earlier = q < p;
        dup |= (earlier & (uint32_t)(qp == pp)) | ((earlier & (uint32_t)(qa == pa)) << 1);
        dup |= ((uint32_t)(qp <= pp) & (uint32_t)(qa >= pa) & ((uint32_t)(qp < pp) | (uint32_t)(qa > pa) | earlier)) << 2;
      }
    }
    dup = group8_or(dup);
    if (p < F && sub == 0) { S.firstP[p] = !(dup & 1u); S.firstA[p] = !(dup & 2u); S.on_stair[p] = !(dup & 4u); }
  }
  if (tid == 0) { S.ks = 0; S.ka = 0; S.fs = 0; }
  if (tid < 256) { S.rankA[tid] = 0u; S.rankB[tid] = ~0ull; S.stair_at[tid] = 0; S.bcnt[tid] = 0u; }
  if (tid < MAX_ACC_WORDS) S.wbits[tid] = 0u;
  __syncthreads();
  // ... and their ranks
  for (uint32_t p0 = 0; p0 < F; p0 += PB) {
    const uint32_t p = p0 + (tid >> 3);
    uint32_t cnt = 0;                                  // latency rank | accuracy rank << 16
    if (p < F) {
      const uint32_t pp = S.pred[p], pa = S.acc[p];
#pragma unroll 4
      for (uint32_t q = sub; q < F; q += 8)
        cnt += ((uint32_t)S.firstP[q] & (uint32_t)(S.pred[q] < pp)) + (((uint32_t)S.firstA[q] & (uint32_t)(S.acc[q] < pa)) << 16);
    }
    cnt = group8_add(cnt);
    if (p < F && sub == 0) {
      const uint32_t rp = cnt & 0xFFFFu, ra = cnt >> 16;
      S.idxP[p] = (unsigned char)rp;
      S.idxA[p] = (unsigned char)ra;
      S.Pd[rp] = S.pred[p];
      S.Ad[ra] = S.acc[p];
      atomicMax(&S.ks, rp + 1);
      atomicMax(&S.ka, ra + 1);
      if (S.on_stair[p]) { atomicAdd(&S.fs, 1u); S.stair_at[rp] = (uint16_t)(p + 1u); }   // one per latency
      atomicMax(&S.rankA[rp], ((uint32_t)S.acc[p] << 16) | (0xFFFFu - p));       // most accurate, first position
      atomicMin(&S.rankB[ra], ((unsigned long long)S.pred[p] << 32) | p);        // fastest, first position
    }
  }
  __syncthreads();
  const uint32_t Ks = S.ks, Ka = S.ka, Fs = S.fs;
  // what the nearest-miss search reads, as running aggregates over the ranks (three warps, while
  // the others start on the masks): bestA[r] over latency ranks < r, bestB[k] over accuracy ranks
  // >= k, ord_start[r] = stair entries with latency rank < r
  if ((tid >> 5) == 0) warp_prefix_max(S.rankA, S.bestA, Ks);
  if ((tid >> 5) == 1) warp_suffix_min(S.rankB, S.bestB, Ka);
  if ((tid >> 5) == 2) warp_prefix_count(S.stair_at, S.ord_start, Ks);
  // block layout and its place in the image; the atomic that places it is in flight while the
  // masks below are built
  const uint32_t acc_lo = c.acc_lo, nbw = c.nbw;      // the catalog's accuracy window
  const uint32_t width = Ka + 1u;
  const BlockLayout BL = block_layout(F, Ks, Ka, first ? 0u : nbw);
  const SlowLayout SL = slow_layout(F, Ks, Ka);
  unsigned long long placed = 0;
  if (tid == 0) placed = place_block_issue(c, BL.bytes, next == 0u);
  // SLO buckets: larger latencies than the largest SLO asked for so far share bucket 255
  uint32_t bmin, Sh;
  bucket_scale(c, Sh, bmin);
  for (uint32_t i = tid; i < Ks; i += B) {
    const uint32_t b = min(max(float_bits(S.Pd[i]) >> Sh, bmin) - bmin, SLO_BUCKETS - 1);
    atomicAdd(&S.bcnt[b], 1u);
    S.bthr[b] = S.Pd[i];                                 // read only where it is the bucket's only one
  }
  for (uint32_t i = tid; i < Ka; i += B) {
    const uint32_t x = S.Ad[i] - acc_lo, xw = x / ACC_WORD_BITS;
    atomicOr(&S.wbits[xw], 1u << (x - xw * ACC_WORD_BITS));
  }
  // position masks: Lmask[r] = positions whose latency rank is < r, Amask[k] = positions whose
  // accuracy rank is >= k (64 positions per word); T2[r][k] is the first bit of their intersection
  const uint32_t nw = (F + 63u) >> 6;
  for (uint32_t x = tid; x < 2u * 256u * nw; x += B) {
    const uint32_t which = x / (256u * nw), y = x - which * 256u * nw, rk = y / nw, w = y - rk * nw;
    if (rk > (which ? Ka : Ks)) continue;
    unsigned long long m = 0;
    const uint32_t p1 = min(F, 64u * w + 64u);
    for (uint32_t p = 64u * w; p < p1; ++p) {
      const bool in = which ? S.idxA[p] >= rk : S.idxP[p] < rk;
      m |= (unsigned long long)in << (p & 63u);
    }
    (which ? S.Amask : S.Lmask)[w][rk] = m;
  }

  if (tid == 0) {
    uint32_t base = image_var_offset(c.n_tasks, nbw) + place_block_finish(c, placed, BL.bytes, next == 0u);
    if (base + BL.bytes > c.image_capacity || base + BL.t2 >= IMAGE_T2_LIMIT) base = 0xFFFFFFFFu;
    S.base = base;
  }
  __syncthreads();
  const uint32_t base = S.base;
  if (base == 0xFFFFFFFFu) return false;
  unsigned char *blk = c.image + base;
  unsigned char *slow = blk + BL.slow;

  // From here on nothing depends on anything else: thread ranges take one small table each.
  // [lo, lo + n) of the CTA's threads run `body(x)` for x = 0 .. count - 1.
  auto share = [&](uint32_t lo, uint32_t n, uint32_t count, auto body) {
    if (tid >= lo && tid < lo + n)
      for (uint32_t x = tid - lo; x < count; x += n) body(x);
  };

  // SLO records (see common.cuh)
  uint32_t *rec = reinterpret_cast<uint32_t *>(c.image + image_rec_offset(c.n_tasks) + t * REC_STRIDE);
  // one bucket per thread of warps 16-23; lb = latencies in lower buckets: the lower warps'
  // buckets summed by the lanes, then a scan inside the warp
  if (first && tid >= B / 2 && tid < B / 2 + SLO_BUCKETS) {
    const uint32_t j = tid - B / 2, lane = tid & 31u;
    uint32_t below = 0;
    for (uint32_t i = lane; i < (j & ~31u); i += 32) below += S.bcnt[i];
    below = __reduce_add_sync(0xFFFFFFFFu, below);
    const uint32_t cnt = S.bcnt[j], thr = S.bthr[j];
    uint32_t incl = cnt;
#pragma unroll
    for (uint32_t o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += y;
    }
    const uint32_t lb = below + incl - cnt;
    const uint32_t lo = j ? float_bits_floor((bmin + j) << Sh) : 0u;
    const uint32_t next = (bmin + j + 1u) << Sh;
    const uint32_t hi = (j == SLO_BUCKETS - 1 || next >= BITS_OF_2_POW_32) ? 0xFFFFFFFFu : float_bits_floor(next) - 1u;
    uint32_t r = (Ks + 1u) << 24;                                // exact slow path
    if (cnt == 0) {
      r = lb << 24;
    } else if (cnt == 1 && (lo >> 24) == (hi >> 24)) {
      r = thr <= lo ? (lb + 1u) << 24 : (lb << 24) | (0x00FFFFFFu - ((thr - 1u) & 0x00FFFFFFu));
    }
    rec[j] = r;
  }

  // accuracy bitmap with running popcounts: warps 24-27, 128 words a round, same scheme; a
  // first segment's bitmap goes into the fixed part of the image
  uint32_t *bitmap = first ? reinterpret_cast<uint32_t *>(c.image + image_bitmap_offset(c.n_tasks) + t * bitmap_stride(nbw))
                           : reinterpret_cast<uint32_t *>(blk + BL.bitmap);
  if (tid >= 3 * B / 4 && tid < 3 * B / 4 + 128u) {
    const uint32_t lane = tid & 31u;
    for (uint32_t w0 = 0; w0 < nbw; w0 += 128u) {              // uniform over the four warps
      const uint32_t w = w0 + (tid - 3 * B / 4);
      uint32_t below = 0;
      for (uint32_t i = lane; i < (w & ~31u); i += 32) below += __popc(S.wbits[i]);
      below = __reduce_add_sync(0xFFFFFFFFu, below);
      const uint32_t bits = w < nbw ? S.wbits[w] : 0u, pc = __popc(bits);
      uint32_t incl = pc;
#pragma unroll
      for (uint32_t o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += y;
      }
      if (w < nbw) bitmap[w] = ((below + incl - pc) << 24) | bits;
    }
  }

  // what the nearest-miss search reads (aggregated above): position 0xFF stands for "none"
  uint32_t *bestA = reinterpret_cast<uint32_t *>(slow + SL.bestA);
  share(7 * B / 8, B / 16, Ks + 1u, [&](uint32_t r) {
    const uint32_t v = S.bestA[r];                               // highest accuracy among ranks < r
    bestA[r] = v ? (v >> 16) | ((0xFFFFu - (v & 0xFFFFu)) << 16) : 0xFFu << 16;
    slow[SL.ordStart + r] = S.ord_start[r];
  });
  uint2 *bestB = reinterpret_cast<uint2 *>(slow + SL.bestB);
  share(15 * B / 16, B / 16, Ka + 1u, [&](uint32_t k) {
    const unsigned long long v = S.bestB[k];                     // lowest latency among accuracy ranks >= k
    bestB[k] = v == ~0ull ? make_uint2(0u, 0xFFu) : make_uint2((uint32_t)(v >> 32), (uint32_t)v);
  });
  // small copies, after the short loops above
  uint32_t *ids_end = reinterpret_cast<uint32_t *>(blk + BL.t2);   // ids, reversed; slot F holds PENDING
  share(3 * B / 4, B / 8, F + 1u, [&](uint32_t p) { ids_end[-1 - (int)p] = p < F ? S.ids[p] : PENDING; });
  uint2 *walk = reinterpret_cast<uint2 *>(slow + SL.walk);      // the stair entries, ascending latency
  share(7 * B / 8, B / 16, F, [&](uint32_t p) {                // stair entries have distinct latencies
    if (S.on_stair[p]) walk[S.ord_start[S.idxP[p]]] = make_uint2(S.pred[p], (uint32_t)S.acc[p] | (p << 16));
  });
  uint32_t *Pd_g = reinterpret_cast<uint32_t *>(slow + SL.Pd);
  share(15 * B / 16, B / 16, Ks, [&](uint32_t i) { Pd_g[i] = S.Pd[i]; });

  // T2: cell (r, k) = first position whose latency rank is < r and accuracy rank >= k.  The
  // largest table: all threads, after their share of the small ones.
  unsigned char *T2 = blk + BL.t2;
  // consecutive lanes take consecutive cells: the same r (a broadcast) and consecutive k, which
  // the word-major masks serve without bank conflicts
  share(0, B, (Ks + 2u) * width, [&](uint32_t cell) {
    const uint32_t r = cell / width, k = cell - r * width;
    uint32_t pos = F;
    if (r >= 1 && r <= Ks)
      for (uint32_t w = 0; w < nw; ++w) {
        const unsigned long long m = S.Lmask[w][r] & S.Amask[w][k];
        if (m) { pos = 64u * w + (uint32_t)__ffsll((long long)m) - 1u; break; }
      }
    T2[cell] = (unsigned char)pos;
  });

  if (tid == 0) {
    if (first) reinterpret_cast<uint32_t *>(c.image + IMAGE_HDR_OFFSET)[t] = (base + BL.t2) | (width << 24);
    else c.xhdr[xi] = make_uint4(base + BL.t2, width, base + BL.bitmap, 0u);
    c.slow[first ? t : c.n_tasks + xi] = make_uint4(base + BL.slow, F | (Ks << 8) | (Ka << 16), 0u, Fs | (next << 8));
  }
  return true;
}

constexpr uint32_t REBUILD_THREADS = 1024;
// build_index gives fixed warps fixed tables: warps 16-23 one SLO bucket per thread, warps 24-27
// the bitmap words
static_assert(REBUILD_THREADS == 1024 && SLO_BUCKETS == 256, "thread ranges of build_index");
constexpr uint32_t RANK_SORT_MAX = 512;   // tasks up to this size are sorted by counting smaller keys

__global__ void __launch_bounds__(REBUILD_THREADS)
rebuild_kernel(DeviceCatalog c, int advance, uint32_t window_us) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ uint32_t warp_sums[32];
  __shared__ uint32_t s_total, s_inlist, s_ncand, s_nnew;
  __shared__ uint16_t filt[RANK_SORT_MAX], cand[RANK_SORT_MAX], newc[RANK_SORT_MAX];   // small tasks: filter set,
  __shared__ unsigned char in_filt[RANK_SORT_MAX];                // candidates, those of them not in the filter set
  __shared__ IndexScratch S;

  const uint32_t t = blockIdx.x, tid = threadIdx.x, B = blockDim.x;
  const uint32_t base = c.task_off[t];
  const uint32_t V = c.task_off[t + 1] - base;

  // sort size for this task: the power of two that holds it (tasks differ in size)
  uint32_t P = 1;
  while (P < V) P <<= 1;
  // small tasks (each task decides for itself) have, in front of the sort buffers, the attributes
  // packed for the prune (kept a plain offset from the shared array so that the loads stay
  // shared-memory loads)
  const bool small = P <= RANK_SORT_MAX;
  uint4 *attr = reinterpret_cast<uint4 *>(smem_raw);
  unsigned long long *k64 = reinterpret_cast<unsigned long long *>(smem_raw + (small ? 16u * P : 0u));   // cost<<32 | pred
  uint32_t *k32 = reinterpret_cast<uint32_t *>(k64 + P);                         // inv_acc<<16 | local
  unsigned char *keep = reinterpret_cast<unsigned char *>(k32 + P);              // 1 = non-dominated

  // A state-aware catalog has two lists per task: Active variants keyed (cost, pred, 10000-acc,
  // id), then Inactive ones keyed by their combined loading + inference latency, which takes
  // the place of both cost and pred.  Each goes through steps 1-4 on its own.
  unsigned char *region = c.regions + c.reg_off[t];
  unsigned long long *keys_g = reinterpret_cast<unsigned long long *>(region);
  uint32_t *ids_g = reinterpret_cast<uint32_t *>(region + 8u * V);
  uint16_t *loc_g = reinterpret_cast<uint16_t *>(region + 12u * V);
  // small tasks: the previous rebuild's survivors (both lists) are the prune's first filter
  const uint32_t n_filt = small ? min(c.f_len[t], V) : 0u;
  if (small) {
    for (uint32_t i = tid; i < V; i += B) in_filt[i] = 0;
    __syncthreads();
    for (uint32_t i = tid; i < n_filt; i += B) {
      const uint32_t f = min((uint32_t)loc_g[i], V - 1u);
      filt[i] = (uint16_t)f;
      in_filt[f] = 1;
    }
  }
  uint32_t F = 0;                         // entries emitted so far
  const uint32_t n_lists = c.stateful ? 2u : 1u;
  for (uint32_t list = 0; list < n_lists; ++list) {
    __syncthreads();
    if (tid == 0) { s_total = 0; s_inlist = 0; s_ncand = 0; s_nnew = 0; }
    __syncthreads();
    // 1. queue recursion and states (first pass), predicted latency, sort keys
    uint32_t mine = 0;
    for (uint32_t i = tid; i < P; i += B) {
      bool in = false;
      uint32_t cost = 0, lat_key = 0, inv = 0;
      if (i < V) {
        const uint32_t slot = base + i;
        // every load before the first store: the arrays may alias as far as the compiler can
        // tell, and each dependent round trip to memory costs about a microsecond here
        const uint32_t acc = c.s_acc[slot];
        uint32_t st = INFAAS_STATE_ACTIVE, load_lat = 0, pred;
        cost = c.s_cost[slot];
        if (c.stateful) { st = c.s_state[slot]; load_lat = c.s_load_lat[slot]; }
        if (list == 0) {
          const uint32_t lat = c.s_lat[slot];
          const uint32_t batch = c.s_batch[slot];
          uint32_t queued = c.s_queued[slot];
          if (advance) {
            const uint32_t id = c.s_id[slot];
            const unsigned long long served = c.s_served[slot];
            const uint32_t cnt = c.count_by_id[id];
            c.s_served[slot] = served + cnt;
            unsigned long long arrived = (unsigned long long)queued + cnt;
            if (arrived > U32_MAX_) arrived = U32_MAX_;
            unsigned long long drain = (unsigned long long)window_us * batch / lat;
            if (drain > U32_MAX_) drain = U32_MAX_;
            queued = arrived > drain ? (uint32_t)(arrived - drain) : 0u;
            c.s_queued[slot] = queued;
            c.count_by_id[id] = 0;      // not right behind its load: a store to an address whose load is
                                        // still in flight holds up everything behind it (measured: 4 us)
            if (c.stateful) {
              // loaded by its first queries; at peak throughput while a backlog remains
              if (st == INFAAS_STATE_INACTIVE && cnt > 0) st = INFAAS_STATE_ACTIVE;
              if (st == INFAAS_STATE_ACTIVE || st == INFAAS_STATE_OVERLOADED)
                st = queued > 0 ? INFAAS_STATE_OVERLOADED : INFAAS_STATE_ACTIVE;
              c.s_state[slot] = (unsigned char)st;
            }
          }
          unsigned long long p = (unsigned long long)lat + (unsigned long long)queued * lat / batch;
          pred = p > U32_MAX_ ? U32_MAX_ : (uint32_t)p;
          c.s_pred[slot] = pred;
        } else {
          pred = c.s_pred[slot];
        }
        in = true;
        lat_key = pred; inv = 10000u - acc;
        if (c.stateful) {
          in = st == (list == 0 ? INFAAS_STATE_ACTIVE : INFAAS_STATE_INACTIVE);
          if (list == 1) {
            const unsigned long long e = (unsigned long long)pred + load_lat;
            cost = lat_key = e > U32_MAX_ ? U32_MAX_ : (uint32_t)e;
          }
        }
      }
      if (in) {
        k64[i] = ((unsigned long long)cost << 32) | lat_key;
        k32[i] = (inv << 16) | i;
        if (small) attr[i] = make_uint4(cost, lat_key, inv, i);
        ++mine;
      } else {
        k64[i] = ~0ull;
        k32[i] = ~0u;
        if (small && i < V) attr[i] = make_uint4(~0u, ~0u, ~0u, i);   // in neither comparison
      }
    }
    mine = __reduce_add_sync(0xFFFFFFFFu, mine);
    if ((tid & 31) == 0 && mine) atomicAdd(&s_inlist, mine);
    __syncthreads();
    const uint32_t Vl = s_inlist;           // variants in this list before the prune

    uint32_t my_kept = 0;
    if (small) {
      // 3 (small tasks, before any sort).  q dominates p iff cost_q <= cost_p, pred_q <= pred_p,
      // acc_q >= acc_p and it differs in some attribute or has the smaller id -- which, given
      // the three inequalities, is the same as its key (cost, pred, 10000-acc, local index)
      // being smaller.  Two rounds.  First every entry is tested against a filter set only,
      // the survivors of the previous rebuild: whatever one of them dominates is gone, whatever
      // set is used.  Every non-dominated entry is among the entries that are left, and,
      // dominance being transitive, each dominated one is dominated by one of those; against the
      // ones inside the filter set it has been tested already, so the second round tests the
      // entries that are left against those of them outside the filter set.  The load moves
      // little from window to window, so these are few.  G lanes share an entry's comparisons
      // in the first round.
      const uint32_t G = min(32u, B / P), p = tid / G, sidx = tid % G;
      uint32_t dom = 0;
      if (p < V) {
        const uint4 a = attr[p];
        if (a.z == ~0u) dom = 1;                         // not in this list
        else {
#pragma unroll 4
          for (uint32_t j = sidx; j < n_filt; j += G) {    // no branch: the loads of several trips overlap
            const uint4 b = attr[filt[j]];                 // (cost, pred, 10000 - acc, local index)
            dom |= dominates(b, a);
          }
        }
      }
      for (uint32_t o = G >> 1; o; o >>= 1) dom |= __shfl_xor_sync(0xFFFFFFFFu, dom, o);   // lane-aligned groups
      {
        const bool is_cand = p < V && sidx == 0 && !dom;
        if (p < V && sidx == 0) keep[p] = !dom;
        const unsigned m = __ballot_sync(0xFFFFFFFFu, is_cand);   // one append per warp, in any order
        uint32_t at = 0;
        if (m && (tid & 31u) == (uint32_t)__ffs(m) - 1u) at = atomicAdd(&s_ncand, (uint32_t)__popc(m));
        at = __shfl_sync(0xFFFFFFFFu, at, m ? __ffs(m) - 1 : 0);
        if (is_cand) cand[at + __popc(m & ((1u << (tid & 31u)) - 1u))] = (uint16_t)p;
        // candidates outside the filter set: the only ones the first round has not tested the others against
        const bool is_new = is_cand && !in_filt[p];
        const unsigned mn = __ballot_sync(0xFFFFFFFFu, is_new);
        uint32_t an = 0;
        if (mn && (tid & 31u) == (uint32_t)__ffs(mn) - 1u) an = atomicAdd(&s_nnew, (uint32_t)__popc(mn));
        an = __shfl_sync(0xFFFFFFFFu, an, mn ? __ffs(mn) - 1 : 0);
        if (is_new) newc[an + __popc(mn & ((1u << (tid & 31u)) - 1u))] = (uint16_t)p;
      }
      __syncthreads();
      const uint32_t R = s_ncand, Nn = s_nnew;
      for (uint32_t x = tid; x < R * Nn; x += B) {
        const uint32_t ip = x / Nn, pp = cand[ip], qq = newc[x - ip * Nn];
        if (dominates(attr[qq], attr[pp])) keep[pp] = 0;   // several writers, one value
      }
      __syncthreads();
      if (tid < V) my_kept = keep[tid];
    } else {
      // 2. bitonic sort of P keys, ascending in (cost, pred, 10000-acc, local index); what is
      // not in this list sorts behind it
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
      // One entry per warp at a time: its 32 lanes scan the earlier entries 32 at a time and stop
      // at the first chunk that holds a dominator (a survivor costs p / 32 trips of the whole
      // warp instead of p trips of one lane).
      for (uint32_t p = tid >> 5; p < V; p += B >> 5) {       // uniform per warp
        bool kp = p < Vl;
        if (kp) {
          const uint32_t pred_p = (uint32_t)k64[p], inv_p = k32[p] >> 16;
          for (uint32_t q0 = 0; q0 < p; q0 += 32) {         // from p - 1 down: a dominator tends to cost
            const uint32_t back = q0 + (tid & 31u);         // about as much as the entry itself
            const uint32_t q = p - 1u - min(back, p - 1u);
            const bool dom = back < p && (uint32_t)k64[q] <= pred_p && (k32[q] >> 16) <= inv_p;
            if (__any_sync(0xFFFFFFFFu, dom)) { kp = false; break; }
          }
        }
        if ((tid & 31u) == 0) { keep[p] = kp; my_kept += kp; }
      }
    }
    __syncthreads();
    my_kept = __reduce_add_sync(0xFFFFFFFFu, my_kept);
    if ((tid & 31) == 0 && my_kept) atomicAdd(&s_total, my_kept);
    __syncthreads();
    const uint32_t Fl = s_total;

    // 4. into the task's region (scan order, behind the earlier list): keys, ids, local indices
    auto emit = [&](uint32_t pos, unsigned long long v64, uint32_t v32) {   // position pos of this list
      const uint32_t pred_p = (uint32_t)v64, acc = 10000u - (v32 >> 16);
      const uint32_t id = c.s_id[base + (v32 & 0xFFFFu)];
      keys_g[F + pos] = ((unsigned long long)acc << 32) | pred_p;
      ids_g[F + pos] = id;
      loc_g[F + pos] = (uint16_t)(v32 & 0xFFFFu);
      if (F + pos < INDEX_MAX_F) { S.ids[F + pos] = id; S.pred[F + pos] = pred_p; S.acc[F + pos] = (uint16_t)acc; }   // first segment
    };
    if (!small) {
      uint32_t kept_so_far = 0;
      for (uint32_t p0 = 0; p0 < V; p0 += B) {      // uniform trip count
        const uint32_t p = p0 + tid;
        const bool kp = p < V && keep[p];
        uint32_t total;
        const uint32_t pos = kept_so_far + block_excl_scan_flag(kp, warp_sums, total);
        if (kp) emit(pos, k64[p], k32[p]);
        kept_so_far += total;
      }
    } else {
      // 2 (small tasks): the survivors' list positions by counting smaller keys among the
      // second round's candidates, of which the survivors are most
      const uint32_t R = s_ncand;
      uint32_t PR = 1;
      while (PR < R) PR <<= 1;
      const uint32_t G = min(32u, B / PR), i = tid / G, sidx = tid % G;
      uint32_t rank = 0;
      unsigned long long a64 = 0;
      uint32_t a32 = 0;
      bool mine_kept = false;
      if (i < R) {
        const uint32_t pp = cand[i];
        mine_kept = keep[pp];
        a64 = k64[pp]; a32 = k32[pp];
        if (mine_kept) {
#pragma unroll 4
          for (uint32_t j = sidx; j < R; j += G) {
            const uint32_t qq = cand[j];
            rank += (uint32_t)keep[qq] & (uint32_t)key_less(k64[qq], k32[qq], a64, a32);
          }
        }
      }
      for (uint32_t o = G >> 1; o; o >>= 1) rank += __shfl_xor_sync(0xFFFFFFFFu, rank, o);
      if (mine_kept && sidx == 0) emit(rank, a64, a32);
    }
    __syncthreads();
    F += Fl;
  }
  bool indexed = F > 0;
  bool counted = false;                       // has this CTA made its last allocation?
  // index the list -- the two lists of a state-aware catalog count as one, the Inactive entries
  // behind the Active ones: "first position that meets both requirements, else the smallest
  // distance at the lowest position" is all the index knows about order -- segment by segment
  // (INDEX_MAX_F positions each; almost always one)
  if (indexed) {
    const uint32_t nseg = (F + INDEX_MAX_F - 1u) / INDEX_MAX_F, x0 = c.seg_base[t];
    for (uint32_t sg = 0; sg < nseg && indexed; ++sg) {
      const uint32_t off = sg * INDEX_MAX_F, Fseg = min(INDEX_MAX_F, F - off);
      if (sg) {                                   // later segments: back from the task's region
        __syncthreads();
        for (uint32_t i = tid; i < Fseg; i += B) {
          const unsigned long long e = keys_g[off + i];
          S.ids[i] = ids_g[off + i]; S.pred[i] = (uint32_t)e; S.acc[i] = (uint16_t)(e >> 32);
        }
        __syncthreads();
      }
      indexed = build_index(c, t, Fseg, S, sg ? x0 + sg - 1u : 0xFFFFFFFFu, sg + 1u < nseg ? x0 + sg + 1u : 0u);
      counted = sg + 1u == nseg;
    }
  }
  if (!counted && tid == 0) place_block_finish(c, place_block_issue(c, 0u, true), 0u, true);   // nothing (more) to place
  if (!indexed) {
    // no index: every query of this task reads "none"
    write_dummy_task(c, t);
    if (tid == 0) c.slow[t] = make_uint4(0u, 0u, F == 0 ? TASK_FLAG_INVALID : TASK_FLAG_NOT_INDEXED, 0u);
  }
  if (t == 0) {
    // entry n_tasks (queries whose task is out of range), the dummy block, and the bucket scale
    // every CTA has used, for the selection kernel
    write_dummy_task(c, c.n_tasks);
    if (tid < IMAGE_DUMMY_BYTES / 4u) reinterpret_cast<uint32_t *>(c.image)[tid] = tid == 3 ? PENDING : 0u;
    if (tid == 0) {
      uint32_t Sh, bmin;
      bucket_scale(c, Sh, bmin);
      c.image_hdr[1] = (127u - Sh) << 23;
      c.image_hdr[2] = __float_as_uint(-(float)bmin);
    }
  }
  if (tid == 0) c.f_len[t] = F;
}

}  // namespace

constexpr uint32_t TALLY_SMEM_MAX_VARIANTS = 49152;   // 192 KB of bins
constexpr uint32_t TALLY_SMEM_MAX_PARTS = 8;           // beyond this many id ranges: global atomics
constexpr uint64_t TALLY_SMEM_MIN_N = 1u << 18;        // below this the zero/flush passes cost more than they save

cudaError_t launch_tally(const DeviceCatalog &c, const uint32_t *d_decision, uint64_t n,
                         int sm_count, cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  const uint32_t parts = (c.n_variants + TALLY_SMEM_MAX_VARIANTS - 1) / TALLY_SMEM_MAX_VARIANTS;
  if (n >= TALLY_SMEM_MIN_N && parts <= TALLY_SMEM_MAX_PARTS) {
    const uint32_t bins = ((c.n_variants + parts - 1) / parts + 3u) & ~3u;
    const size_t smem = (size_t)(bins + 32) * 4;                 // 32 spare bins
    // one CTA of 1024 threads per SM: half as many histograms to clear and flush as two of 512
    uint64_t want = ((n >> 2) + TALLY_SMEM_THREADS * 8 - 1) / (TALLY_SMEM_THREADS * 8);
    uint64_t shares = (uint64_t)sm_count / parts;              // CTAs per id range
    if (shares > want) shares = want;
    if (shares < 1) shares = 1;
    tally_smem_kernel<<<(uint32_t)(shares * parts), TALLY_SMEM_THREADS, smem, stream>>>(
        d_decision, n, c.n_variants, bins, parts, c.count_by_id, c.counters);
    return cudaGetLastError();
  }
  uint64_t want = ((n >> 2) + 255) / 256;
  const uint64_t most = (uint64_t)sm_count * 8;
  uint32_t grid = (uint32_t)(want < 1 ? 1 : (want > most ? most : want));
  tally_kernel<<<grid, 256, 0, stream>>>(d_decision, n, c.n_variants, c.count_by_id, c.counters);
  return cudaGetLastError();
}

cudaError_t prepare_rebuild_kernel() {
  cudaError_t e = cudaFuncSetAttribute(tally_smem_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)((TALLY_SMEM_MAX_VARIANTS + 32) * 4));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(rebuild_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)REBUILD_MAX_SMEM);
}

cudaError_t launch_rebuild(const DeviceCatalog &c, bool advance_queues, uint32_t window_us,
                           cudaStream_t stream) {
  uint32_t P = 1;
  while (P < c.max_task_variants) P <<= 1;
  // sort buffers of the largest task (13 bytes per padded entry); a small task needs 29 bytes per
  // padded entry (packed attributes in front), at most for RANK_SORT_MAX entries
  const uint32_t Ps = P < RANK_SORT_MAX ? P : RANK_SORT_MAX;
  size_t smem = (size_t)P * 13;
  if (smem < (size_t)Ps * 29 + 32) smem = (size_t)Ps * 29 + 32;
  rebuild_kernel<<<c.n_tasks, REBUILD_THREADS, smem, stream>>>(c, advance_queues ? 1 : 0, window_us);
  return cudaGetLastError();
}

}  // namespace infaas
