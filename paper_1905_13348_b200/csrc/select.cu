// Selection kernel: for each query (task, latency SLO, minimum accuracy) pick the cheapest
// variant of the task that meets both requirements, else flag the nearest miss
// (Section 4.1 of the paper, "Case I: on arrival of a query"; cost objective as in the
// worked example of Section 2.2).
//
// Each task's scan list is sorted by (cost, pred_lat, -acc, id) and pruned to non-dominated
// variants, so the answer for a feasible query is the FIRST list position that meets both
// requirements.  Instead of walking the list, a thread ranks the query's SLO among the
// list's distinct latencies (one bucket record, one add) and its minimum accuracy among
// the list's distinct accuracies (one bitmap word, one popcount) and reads the answer's
// position from a small per-task table indexed by the two ranks (layout in common.cuh):
// five shared-memory loads per query, no loop, no compare.  The packed image of all tasks
// is staged in shared memory once per CTA with bulk asynchronous copies (TMA, mbarrier
// completion); queries stream through with 128-bit loads and stores, four per thread and
// iteration.  Queries the tables cannot answer (nothing feasible, an SLO bucket holding
// several latencies, a task without index) come out of the fast path as PENDING; they are
// parked per warp in shared memory with their data and resolved 32 at a time.
#include "common.cuh"

namespace infaas {

namespace {

constexpr int SELECT_THREADS = 1024;
constexpr int SELECT_WARPS = SELECT_THREADS / 32;
constexpr uint32_t WARP_TILE = 128;              // queries per warp and iteration
constexpr uint32_t PARK_CAP = 64;                // parked queries per warp (flushed at 32)
constexpr uint32_t PARK_BYTES = SELECT_WARPS * PARK_CAP * 16;
constexpr uint32_t STAGE_CHUNK = 32768;          // bytes per bulk copy
constexpr uint32_t STAGE_POLL_LIMIT = 1u << 22;  // bounded wait on the staging barrier
constexpr uint32_t MAX_SPAN = 1u << 31;          // queries per CTA (offsets are 32-bit)

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

// Start staging `bytes` (multiple of 16) from global `src` (16-byte aligned) into shared
// `dst`; completion is signalled on `mbar`.
__device__ __forceinline__ void stage_begin(unsigned char *dst, const unsigned char *src, uint32_t bytes,
                                            unsigned long long *mbar) {
  const uint32_t bar = smem_u32(mbar);
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
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
  __syncthreads();   // the barrier is initialised before anyone polls it
}

// Wait for the staged bytes.  Returns false (all threads) if they did not arrive within
// the poll limit.
__device__ __forceinline__ bool stage_wait(unsigned long long *mbar) {
  const uint32_t bar = smem_u32(mbar);
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

// The image, read either from shared memory (32-bit addresses, ld.shared) or from global
// memory (read-only path).  Offsets are bytes from the start of the image.
struct SharedImage {
  uint32_t base;
  __device__ __forceinline__ uint32_t u8(uint32_t off) const {
    uint32_t v; asm("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(base + off)); return v;
  }
  __device__ __forceinline__ uint32_t u32(uint32_t off) const {
    uint32_t v; asm("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(base + off)); return v;
  }
  __device__ __forceinline__ uint2 v2(uint32_t off) const {
    uint2 v; asm("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(base + off)); return v;
  }
};

struct GlobalImage {
  const unsigned char *base;
  __device__ __forceinline__ uint32_t u8(uint32_t off) const { return __ldg(base + off); }
  __device__ __forceinline__ uint32_t u32(uint32_t off) const {
    return __ldg(reinterpret_cast<const uint32_t *>(base + off));
  }
  __device__ __forceinline__ uint2 v2(uint32_t off) const {
    return __ldg(reinterpret_cast<const uint2 *>(base + off));
  }
};

// floor(a / 24) for a < 2^16 as the high half of a product (multiply pipe).
__device__ __forceinline__ uint32_t div24(uint32_t a) { return __umulhi(a, 178956971u); }

// What the lookups need that does not depend on the task: the bucket scale the last rebuild
// used, the catalog's accuracy window, and where the fixed tables sit in the image.
struct Fixed {
  float scale, neg_bmin;      // bucket of an SLO: floor(bits(slo) * scale + neg_bmin), saturated to 0..255
  uint32_t n_tasks;
  uint32_t rec_off;           // image offset of the SLO records
  uint32_t bm_off;            // image offset of the first tasks' bitmaps, less 4 * (acc_lo / 24)
  uint32_t bm_stride;         // bytes of one bitmap
  uint32_t acc_lo, acc_hi;    // accuracy window, both ends included
};
// `hdr`: the words the last rebuild published (image bytes, bucket scale, -bmin).
__device__ __forceinline__ Fixed make_fixed(const DeviceCatalog &c, const uint4 hdr) {
  Fixed f;
  f.scale = __uint_as_float(hdr.y);
  f.neg_bmin = __uint_as_float(hdr.z);
  f.n_tasks = c.n_tasks;
  f.rec_off = image_rec_offset(c.n_tasks);
  f.bm_off = image_bitmap_offset(c.n_tasks) - 4u * (c.acc_lo / ACC_WORD_BITS);
  f.bm_stride = bitmap_stride(c.nbw);
  f.acc_lo = c.acc_lo;
  f.acc_hi = c.acc_lo + ACC_WORD_BITS * c.nbw - 1u;
  return f;
}

// k = #{distinct list accuracies < min_acc} from a bitmap with running popcounts whose word
// for accuracy acc_lo sits at image offset bm0 + 4 * (acc_lo / 24).
template <bool Clamped, class Img>
__device__ __forceinline__ uint32_t acc_rank(const Img &img, const Fixed &fx, uint32_t bm0, uint32_t min_acc) {
  const uint32_t a = Clamped ? min_acc : min(max(min_acc, fx.acc_lo), fx.acc_hi);
  const uint32_t w = div24(a);
  const uint32_t word = img.u32(bm0 + (w << 2));
  const uint32_t below = word & ((1u << (a - w * ACC_WORD_BITS)) - 1u);   // prefix byte masked off: shift < 24
  return __umulhi(word, 1u << 8) + __popc(below);
}

// Fast path, straight-line: five loads, no compare.  Returns the variant id, or PENDING
// when the tables cannot answer (nothing feasible, an SLO bucket with several latencies,
// a task without index or out of range).
// `Clamped`: the caller has already limited the task to n_tasks and the accuracy to the window.
template <bool Clamped, class Img>
__device__ __forceinline__ uint32_t decide_fast(const Img &img, const Fixed &fx, uint32_t task, uint32_t slo,
                                                uint32_t min_acc) {
  const uint32_t t = Clamped ? task : min(task, fx.n_tasks);
  const uint32_t h = img.u32(IMAGE_HDR_OFFSET + (t << 2));
  // bucket of the SLO: floor(bits(slo) * 2^-S) - bmin, saturated to 0..255 by the conversion
  const float code = __uint2float_rz(__float_as_uint(__uint2float_rz(slo)));
  uint32_t j;
  asm("cvt.rmi.sat.u8.f32 %0, %1;" : "=r"(j) : "f"(fmaf(code, fx.scale, fx.neg_bmin)));
  const uint32_t rec = img.u32(fx.rec_off + t * REC_STRIDE + (j << 2));
  const uint32_t r = __umulhi(rec + (slo & 0x00FFFFFFu), 1u << 8);
  const uint32_t k = acc_rank<Clamped>(img, fx, fx.bm_off + t * fx.bm_stride, min_acc);
  const uint32_t t2 = h & 0x00FFFFFFu, width = h >> 24;
  const uint32_t pos = img.u8(t2 + r * width + k);
  return img.u32(t2 - 4u - (pos << 2));
}

// Slow path for a parked query.
//   Indexed list: exact ranks (binary search over the distinct latencies), then T2.  If
//   nothing is feasible the nearest miss is the entry smallest in (d, position), with
//   d = 10^4 * max(0, pred - slo) + slo * max(0, min_acc - acc) in 64 bits -- position
//   order is (cost, pred_lat, -acc, id) order.  Entries that meet the SLO all miss the
//   accuracy, the best of them is the one with the highest accuracy (bestA); entries that
//   meet the accuracy all miss the SLO, the best being the one with the lowest latency
//   (bestB); an entry that misses both can only win with accuracy above bestA's and latency
//   not above bestB's, and then only if no other entry is at least as fast and at least as
//   accurate (for slo > 0 such an entry is strictly closer), so only those "stair" entries
//   are walked, in latency order, until the latency overshoot alone exceeds the best
//   distance so far.  For slo = 0 the accuracy term vanishes: the answer is the fastest entry.
//   A list longer than INDEX_MAX_F is a chain of segments, each with tables of its own: the
//   first segment with a feasible entry answers; otherwise the closest of the segments' misses.
//   List without index: walk it in global memory, for a feasible entry, then for the distance.
// One segment of a task's list (at most INDEX_MAX_F consecutive positions with their own
// tables): returns the id of its first feasible entry, or PENDING after folding the
// segment's nearest miss into (best, best_id); a later segment wins only with a strictly
// smaller distance, since its positions are all higher.
template <class Img>
__device__ __forceinline__ uint32_t slow_segment(const Img &img, const Fixed &fx, const uint4 sl, uint32_t t2,
                                                 uint32_t width, uint32_t bm0, uint32_t slo, uint32_t min_acc,
                                                 unsigned long long &best, uint32_t &best_id) {
  const uint32_t F = sl.y & 0xFFu, Ks = (sl.y >> 8) & 0xFFu, Ka = sl.y >> 16, Fs = sl.w & 0xFFu;
  const SlowLayout SL = slow_layout(F, Ks, Ka);
  const uint32_t so = sl.x;
  uint32_t r = 0;                                            // r = #{Pd <= slo}
#pragma unroll
  for (uint32_t step = 128; step; step >>= 1) {
    const uint32_t probe = r + step;
    if (probe <= Ks && img.u32(so + SL.Pd + ((probe - 1u) << 2)) <= slo) r = probe;
  }
  const uint32_t k = acc_rank<false>(img, fx, bm0, min_acc);
  const uint32_t pos = img.u8(t2 + r * width + k);
  if (pos < F) return img.u32(t2 - 4u - (pos << 2));
  unsigned long long mine = ~0ull;        // this segment's nearest miss
  uint32_t mine_p = 0;
  if (slo == 0u) {                        // the accuracy term vanishes: the fastest entry
    const uint2 Bv = img.v2(so + SL.bestB);
    mine = (unsigned long long)Bv.x * 10000ull;
    mine_p = Bv.y;
  } else {
    uint32_t acc_floor = 0;               // candidates that miss both need accuracy >= this
    uint32_t pred_cap = 0xFFFFFFFFu;      // ... and latency <= this
    if (r > 0) {                          // some entry meets the SLO (and misses the accuracy)
      const uint32_t A = img.u32(so + SL.bestA + (r << 2));
      mine = (unsigned long long)slo * (min_acc - (A & 0xFFFFu));
      mine_p = A >> 16;
      acc_floor = (A & 0xFFFFu) + 1u;
    }
    if (k < Ka) {                         // some entry meets the accuracy (and misses the SLO)
      const uint2 Bv = img.v2(so + SL.bestB + (k << 3));
      const unsigned long long d = (unsigned long long)(Bv.x - slo) * 10000ull;
      if (d < mine || (d == mine && Bv.y < mine_p)) { mine = d; mine_p = Bv.y; }
      pred_cap = Bv.x;
    }
    for (uint32_t o = img.u8(so + SL.ordStart + r); o < Fs; ++o) {   // stair entries above the SLO, ascending
      const uint2 e = img.v2(so + SL.walk + (o << 3));
      if (e.x > pred_cap) break;
      const unsigned long long over = (unsigned long long)(e.x - slo) * 10000ull;
      if (over > mine) break;             // later entries overshoot the SLO even more
      const uint32_t acc = e.y & 0xFFFFu, p = e.y >> 16;
      if (acc >= acc_floor && acc < min_acc) {
        const unsigned long long d = over + (unsigned long long)slo * (min_acc - acc);
        if (d < mine || (d == mine && p < mine_p)) { mine = d; mine_p = p; }
      }
    }
  }
  if (mine < best) { best = mine; best_id = img.u32(t2 - 4u - (mine_p << 2)); }
  return PENDING;
}

template <class Img>
__device__ __forceinline__ uint32_t decide_slow(const Img &img, const DeviceCatalog &c, const Fixed &fx, uint32_t task,
                                                uint32_t slo, uint32_t min_acc) {
  if (task >= c.n_tasks) return INFAAS_INVALID;
  uint4 sl = __ldg(c.slow + task);
  if (sl.z & TASK_FLAG_INVALID) return INFAAS_INVALID;
  unsigned long long best = ~0ull;
  uint32_t best_p = 0;
  if (!(sl.z & TASK_FLAG_NOT_INDEXED)) {
    // the list's segments in order: the first has its header word and bitmap in the fixed part
    // of the image, the others (lists longer than INDEX_MAX_F) a header in global memory
    const uint32_t h = img.u32(IMAGE_HDR_OFFSET + (task << 2));
    uint32_t t2 = h & 0x00FFFFFFu, width = h >> 24, bm0 = fx.bm_off + task * fx.bm_stride;
    for (;;) {
      const uint32_t d = slow_segment(img, fx, sl, t2, width, bm0, slo, min_acc, best, best_p);
      if (d != PENDING) return d;
      const uint32_t next = sl.w >> 8;                       // 1 + index of the next segment
      if (next == 0u) break;
      sl = __ldg(c.slow + c.n_tasks + next - 1u);
      const uint4 xh = __ldg(c.xhdr + next - 1u);
      t2 = xh.x; width = xh.y; bm0 = xh.z - 4u * (fx.acc_lo / ACC_WORD_BITS);
    }
    return INFAAS_NO_FEASIBLE | best_p;
  }
  const uint32_t F = __ldg(c.f_len + task);
  const uint32_t V = __ldg(c.task_off + task + 1) - __ldg(c.task_off + task);
  const unsigned char *region = c.regions + __ldg(c.reg_off + task);
  const unsigned long long *keys = reinterpret_cast<const unsigned long long *>(region);
  const uint32_t *ids = reinterpret_cast<const uint32_t *>(region + 8u * V);
  for (uint32_t i = 0; i < F; ++i) {
    const unsigned long long e = __ldg(keys + i);
    if ((uint32_t)e <= slo && (uint32_t)(e >> 32) >= min_acc) return __ldg(ids + i);
  }
  for (uint32_t i = 0; i < F; ++i) {
    const unsigned long long e = __ldg(keys + i);
    const uint32_t pred = (uint32_t)e, acc = (uint32_t)(e >> 32);
    const unsigned long long d = (unsigned long long)(pred > slo ? pred - slo : 0u) * 10000ull +
                                 (unsigned long long)slo * (min_acc > acc ? min_acc - acc : 0u);
    if (d < best) { best = d; best_p = i; }
  }
  return INFAAS_NO_FEASIBLE | __ldg(ids + best_p);
}

struct Queries {
  const uint16_t *__restrict__ task;
  const uint32_t *__restrict__ slo;
  const uint16_t *__restrict__ min_acc;
  uint32_t *__restrict__ decision;
};

// A warp's park list in shared memory, one 16-byte entry per parked query: offset of the
// query from the CTA's first query, SLO, task | min_acc << 16, and a spare word.
struct Park {
  uint4 *e;
  uint32_t cnt;
};

// Per-thread sums of the decisions tallied by the fused form of the kernel (feasible, nothing
// feasible, invalid), added to the catalog's counters at the end.
struct Tallies {
  uint32_t feas = 0, nofeas = 0, inval = 0;
};

// Tally one decision per lane into the per-variant counts (Section 4.2.2: the load a variant
// serves is tracked from the queries it is given): lanes of the warp that hold the same variant
// share one atomic.  `live`: this lane holds a final decision.  All lanes call this together.
__device__ __forceinline__ void tally_decision(const DeviceCatalog &c, uint32_t d, bool live, Tallies &tl) {
  const bool feas = live && d < c.n_variants;                 // n_variants < 2^31: bit 31 clear
  const bool inval = live && !feas && (d == INFAAS_INVALID || !(d & INFAAS_NO_FEASIBLE));
  tl.feas += feas;
  tl.inval += inval;
  tl.nofeas += live && !feas && !inval;
  const unsigned fm = __ballot_sync(0xFFFFFFFFu, feas);
  if (feas) {
    const unsigned peers = __match_any_sync(fm, d);
    if ((threadIdx.x & 31u) == (uint32_t)__ffs(peers) - 1u) atomicAdd(&c.count_by_id[d], (uint32_t)__popc(peers));
  }
}

// Resolve the parked queries [first, first + count), count <= 32, one per lane.
template <bool Tally, class Img>
__device__ __forceinline__ void resolve_parked(const Img &img, const DeviceCatalog &c, const Fixed &fx, uint32_t *out,
                                               const Park &pk, uint32_t first, uint32_t count, Tallies &tl) {
  const uint32_t lane = threadIdx.x & 31;
  uint32_t d = 0;
  if (lane < count) {
    const uint4 e = pk.e[first + lane];
    d = decide_slow(img, c, fx, e.z & 0xFFFFu, e.y, e.z >> 16);
    out[e.x] = d;
  }
  if (Tally) {
    __syncwarp();
    tally_decision(c, d, lane < count, tl);
  }
}

// Park the queries a lane holds whose bit is set in `pm` (bit i = i-th of its four
// queries, data in ta[i] / s[i], offset rel + i); flush whenever 32 are waiting.  All
// lanes of the warp call this together.
template <bool Tally, class Img>
__device__ __forceinline__ void park_and_flush(const Img &img, const DeviceCatalog &c, const Fixed &fx, uint32_t *out, Park &pk,
                                               uint32_t pm, uint32_t rel, const uint32_t (&ta)[4],
                                               const uint32_t (&s)[4], Tallies &tl) {
  const uint32_t lane_lt = (1u << (threadIdx.x & 31)) - 1u;
  unsigned m;
  while ((m = __ballot_sync(0xFFFFFFFFu, pm != 0u)) != 0u) {
    if (pm) {
      const uint32_t i = __ffs(pm) - 1u;
      pk.e[pk.cnt + __popc(m & lane_lt)] =
          make_uint4(rel + i, i == 0 ? s[0] : i == 1 ? s[1] : i == 2 ? s[2] : s[3],
                     i == 0 ? ta[0] : i == 1 ? ta[1] : i == 2 ? ta[2] : ta[3], 0u);
      pm &= pm - 1u;
    }
    pk.cnt += __popc(m);
    __syncwarp();
    if (pk.cnt >= 32) {
      pk.cnt -= 32;
      resolve_parked<Tally>(img, c, fx, out, pk, pk.cnt, 32, tl);
      __syncwarp();
    }
  }
}

// `Tally`: also count the decisions per variant (the first half of the load update), for
// batches small enough that a second pass over them would cost more than the atomics here.
template <bool Tally, class Img>
__device__ __forceinline__ void select_body(const Img &img, const DeviceCatalog &c, const Queries &q,
                                            uint64_t q0, uint32_t span, uint4 *park_all, const uint4 hdr,
                                            uint32_t slo_seen, uint2 t4, uint4 s4, uint2 a4) {
  const Fixed fx = make_fixed(c, hdr);
  Tallies tl;
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  Park pk;
  pk.e = park_all + warp * PARK_CAP;
  pk.cnt = 0;
  uint32_t *out = q.decision + q0;
  const uint32_t full_tiles = span / WARP_TILE;
  const uint32_t t_max2 = fx.n_tasks * 0x10001u, a_lo2 = fx.acc_lo * 0x10001u, a_hi2 = fx.acc_hi * 0x10001u;

  // full tiles: 4 consecutive queries per lane, 128-bit loads, next tile prefetched (the
  // first tile was loaded by the caller while the image was being staged)
  uint32_t slo_or = 0;                  // how large the SLOs get: sizes the buckets of later rebuilds
  for (uint32_t tile = warp; tile < full_tiles; tile += SELECT_WARPS) {
    const uint2 t = t4, a = a4;
    const uint4 s = s4;
    slo_or |= s.x | s.y | s.z | s.w;
    const uint32_t next = tile + SELECT_WARPS;
    if (next < full_tiles) {
      const uint64_t i4 = (q0 + (uint64_t)next * WARP_TILE) / 4 + lane;
      t4 = __ldcs(reinterpret_cast<const uint2 *>(q.task) + i4);
      s4 = __ldcs(reinterpret_cast<const uint4 *>(q.slo) + i4);
      a4 = __ldcs(reinterpret_cast<const uint2 *>(q.min_acc) + i4);
    }
    const uint32_t tq[4] = {t.x & 0xFFFFu, t.x >> 16, t.y & 0xFFFFu, t.y >> 16};
    const uint32_t aq[4] = {a.x & 0xFFFFu, a.x >> 16, a.y & 0xFFFFu, a.y >> 16};
    const uint32_t sq[4] = {s.x, s.y, s.z, s.w};
    // tasks limited to n_tasks (the entry of "out of range") and accuracies to the bitmaps'
    // window, two 16-bit values per instruction
    const uint32_t tcx = __vminu2(t.x, t_max2), tcy = __vminu2(t.y, t_max2);
    const uint32_t acx = __vminu2(__vmaxu2(a.x, a_lo2), a_hi2), acy = __vminu2(__vmaxu2(a.y, a_lo2), a_hi2);
    uint4 d;
    d.x = decide_fast<true>(img, fx, tcx & 0xFFFFu, sq[0], acx & 0xFFFFu);
    d.y = decide_fast<true>(img, fx, tcx >> 16, sq[1], acx >> 16);
    d.z = decide_fast<true>(img, fx, tcy & 0xFFFFu, sq[2], acy & 0xFFFFu);
    d.w = decide_fast<true>(img, fx, tcy >> 16, sq[3], acy >> 16);
    const uint32_t rel = tile * WARP_TILE + lane * 4u;
    // PENDING slots are overwritten by the lane that resolves them, after a warp barrier
    __stcs(reinterpret_cast<uint4 *>(out + rel), d);
    if (Tally) {                         // what is PENDING is tallied when it is resolved
      tally_decision(c, d.x, d.x != PENDING, tl);
      tally_decision(c, d.y, d.y != PENDING, tl);
      tally_decision(c, d.z, d.z != PENDING, tl);
      tally_decision(c, d.w, d.w != PENDING, tl);
    }
    // valid ids stay below 2^31, PENDING has bit 31 set
    if (__any_sync(0xFFFFFFFFu, (int)(d.x | d.y | d.z | d.w) < 0)) {
      const uint32_t pm = (d.x >> 31) | ((d.y >> 31) << 1) | ((d.z >> 31) << 2) | ((d.w >> 31) << 3);
      const uint32_t ta[4] = {tq[0] | (aq[0] << 16), tq[1] | (aq[1] << 16), tq[2] | (aq[2] << 16),
                              tq[3] | (aq[3] << 16)};
      __syncwarp();
      park_and_flush<Tally>(img, c, fx, out, pk, pm, rel, ta, sq, tl);
    }
  }
  // ragged tail of the CTA's range (fewer than WARP_TILE queries): one warp, scalar accesses
  const uint32_t tail0 = full_tiles * WARP_TILE;
  if (tail0 < span && warp == full_tiles % SELECT_WARPS) {
    for (uint32_t j = 0; j < WARP_TILE / 32; ++j) {
      const uint32_t rel = tail0 + j * 32u + lane;
      uint32_t d = 0, ta[4] = {0, 0, 0, 0}, sq[4] = {0, 0, 0, 0};
      if (rel < span) {
        const uint64_t i = q0 + rel;
        const uint32_t tk = q.task[i], ac = q.min_acc[i];
        sq[0] = q.slo[i];
        slo_or |= sq[0];
        ta[0] = tk | (ac << 16);
        d = decide_fast<false>(img, fx, tk, sq[0], ac);
        out[rel] = d;
      }
      __syncwarp();
      if (Tally) tally_decision(c, d, rel < span && d != PENDING, tl);
      park_and_flush<Tally>(img, c, fx, out, pk, d >> 31, rel, ta, sq, tl);
    }
  }
  __syncwarp();
  resolve_parked<Tally>(img, c, fx, out, pk, 0, pk.cnt, tl);
  slo_or = __reduce_or_sync(0xFFFFFFFFu, slo_or);
  if (lane == 0 && (slo_or & ~slo_seen)) atomicOr(c.slo_seen, slo_or);
  if (Tally) {
    const uint32_t f = __reduce_add_sync(0xFFFFFFFFu, tl.feas), nf = __reduce_add_sync(0xFFFFFFFFu, tl.nofeas),
                   iv = __reduce_add_sync(0xFFFFFFFFu, tl.inval);
    if (lane == 0) {
      if (f) atomicAdd(&c.counters[0], (unsigned long long)f);
      if (nf) atomicAdd(&c.counters[1], (unsigned long long)nf);
      if (iv) atomicAdd(&c.counters[2], (unsigned long long)iv);
    }
  }
}

template <bool Tally>
__global__ void __launch_bounds__(SELECT_THREADS, 1)
select_kernel(DeviceCatalog c, uint32_t stage_bytes, Queries q, uint64_t n, uint64_t per_cta) {
  extern __shared__ __align__(128) unsigned char smem[];   // [park lists][staged image]
  __shared__ __align__(8) unsigned long long mbar;
  uint4 *park = reinterpret_cast<uint4 *>(smem);
  unsigned char *staged = smem + PARK_BYTES;
  const uint64_t q0 = (uint64_t)blockIdx.x * per_cta;
  if (q0 >= n) return;
  const uint32_t span = (uint32_t)min(n - q0, per_cta);     // <= MAX_SPAN (checked by the launcher)
  // Everything the kernel has to wait for before its first decision starts at once: the staging
  // of `stage_bytes` (what the host planned for: the reserved room or the image buffer, whichever
  // is smaller -- the bytes behind the live image are never looked at), the words the last rebuild
  // published, the SLO mask, and every warp's first tile.
  if (stage_bytes) stage_begin(staged, c.image, stage_bytes, &mbar);
  const uint4 hdr = __ldg(reinterpret_cast<const uint4 *>(c.image_hdr));
  const uint32_t slo_seen = __ldg(c.slo_seen);
  uint2 t4 = make_uint2(0, 0), a4 = make_uint2(0, 0);
  uint4 s4 = make_uint4(0, 0, 0, 0);
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp < span / WARP_TILE) {
    const uint64_t i4 = (q0 + (uint64_t)warp * WARP_TILE) / 4 + lane;
    t4 = __ldcs(reinterpret_cast<const uint2 *>(q.task) + i4);
    s4 = __ldcs(reinterpret_cast<const uint4 *>(q.slo) + i4);
    a4 = __ldcs(reinterpret_cast<const uint2 *>(q.min_acc) + i4);
  }
  // the copy is waited for in any case: the CTA must not end with it in flight
  if (stage_bytes && !stage_wait(&mbar)) {
    if (threadIdx.x == 0) atomicMax(c.err, (uint32_t)DEV_ERR_STAGE_TIMEOUT);
    return;
  }
  if (hdr.x <= stage_bytes) {
    SharedImage img{smem_u32(staged)};
    select_body<Tally>(img, c, q, q0, span, park, hdr, slo_seen, t4, s4, a4);
  } else {
    // the image is larger than what was staged: read it from global memory (L1/L2 resident)
    GlobalImage img{c.image};
    select_body<Tally>(img, c, q, q0, span, park, hdr, slo_seen, t4, s4, a4);
  }
}

}  // namespace

cudaError_t prepare_select_kernel() {
  cudaError_t e = cudaFuncSetAttribute(select_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)SELECT_MAX_SMEM);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)SELECT_MAX_SMEM);
}

uint32_t select_image_smem(uint32_t image_smem) {
  if (image_smem + PARK_BYTES > SELECT_MAX_SMEM) image_smem = (SELECT_MAX_SMEM - PARK_BYTES) & ~15u;
  return image_smem;
}

cudaError_t launch_select(const DeviceCatalog &c, const uint16_t *d_task, const uint32_t *d_slo,
                          const uint16_t *d_min_acc, uint64_t n, uint32_t *d_decision,
                          int sm_count, uint32_t image_smem, bool tally, cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  image_smem = select_image_smem(image_smem);
  // one CTA per SM; every CTA takes one contiguous range, a multiple of the warp tile
  const uint64_t tiles = (n + WARP_TILE - 1) / WARP_TILE;
  uint64_t grid = (uint64_t)sm_count;
  if (grid > tiles) grid = tiles;
  uint64_t per_cta = (tiles + grid - 1) / grid * WARP_TILE;
  if (per_cta > MAX_SPAN) per_cta = MAX_SPAN;               // very large batches: more CTAs than SMs
  grid = (n + per_cta - 1) / per_cta;
  if (grid > 0x7FFFFFFFull) return cudaErrorInvalidValue;
  Queries q{d_task, d_slo, d_min_acc, d_decision};
  const uint32_t stage_bytes = (image_smem < c.image_capacity ? image_smem : c.image_capacity) & ~15u;
  if (tally)
    select_kernel<true><<<(uint32_t)grid, SELECT_THREADS, image_smem + PARK_BYTES, stream>>>(c, stage_bytes, q, n, per_cta);
  else
    select_kernel<false><<<(uint32_t)grid, SELECT_THREADS, image_smem + PARK_BYTES, stream>>>(c, stage_bytes, q, n, per_cta);
  return cudaGetLastError();
}

}  // namespace infaas
