// Selection kernel: for each query (task, latency SLO, minimum accuracy) pick the cheapest
// variant of the task that meets both requirements, else flag the nearest miss
// (Section 4.1 of the paper, "Case I: on arrival of a query"; cost objective as in the
// worked example of Section 2.2).
//
// Each task's scan list is sorted by (cost, pred_lat, -acc, id) and pruned to non-dominated
// variants, so the answer for a feasible query is the FIRST list position that meets both
// requirements.  Instead of walking the list, a thread ranks the query's SLO among the
// list's distinct latencies (one bucket record, one comparison) and its minimum accuracy
// among the list's distinct accuracies (one bitmap word, one popcount) and reads the
// answer's position from a small per-task table indexed by the two ranks (layout in
// common.cuh): five shared-memory loads per query, no loop.  The packed image of all
// tasks is staged in shared memory once per CTA with bulk asynchronous copies (TMA,
// mbarrier completion); queries stream through with 128-bit loads and stores, four per
// thread and iteration.  Queries without a feasible variant (and those of a task whose list
// is too long for the index) are parked in a per-warp list and resolved 32 at a time with
// all lanes busy.
#include "common.cuh"

namespace infaas {

namespace {

constexpr int SELECT_THREADS = 1024;
constexpr int SELECT_WARPS = SELECT_THREADS / 32;
constexpr uint32_t WARP_TILE = 128;              // queries per warp and iteration
constexpr uint32_t PARK_CAP = 32 + WARP_TILE;    // parked queries per warp
constexpr uint32_t PARK_BYTES = SELECT_WARPS * PARK_CAP * 4;
constexpr uint32_t STAGE_CHUNK = 32768;          // bytes per bulk copy
constexpr uint32_t STAGE_POLL_LIMIT = 1u << 22;  // bounded wait on the staging barrier
constexpr uint32_t PENDING = 0xFFFFFFFEu;        // never a valid decision (ids stop at 2^31-3)

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

// Stage `bytes` (multiple of 16) from global `src` (16-byte aligned) into shared `dst`.
// Returns false if the copy did not complete within the poll limit.
__device__ __forceinline__ bool stage_image(unsigned char *dst, const unsigned char *src,
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
  __device__ __forceinline__ uint32_t u16(uint32_t off) const {
    uint32_t v; asm("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(base + off)); return v;
  }
  __device__ __forceinline__ uint2 v2(uint32_t off) const {
    uint2 v; asm("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(base + off)); return v;
  }
  __device__ __forceinline__ uint4 v4(uint32_t off) const {
    uint4 v;
    asm("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(base + off));
    return v;
  }
};

struct GlobalImage {
  const unsigned char *base;
  __device__ __forceinline__ uint32_t u8(uint32_t off) const { return __ldg(base + off); }
  __device__ __forceinline__ uint32_t u32(uint32_t off) const {
    return __ldg(reinterpret_cast<const uint32_t *>(base + off));
  }
  __device__ __forceinline__ uint32_t u16(uint32_t off) const {
    return __ldg(reinterpret_cast<const uint16_t *>(base + off));
  }
  __device__ __forceinline__ uint2 v2(uint32_t off) const {
    return __ldg(reinterpret_cast<const uint2 *>(base + off));
  }
  __device__ __forceinline__ uint4 v4(uint32_t off) const {
    return __ldg(reinterpret_cast<const uint4 *>(base + off));
  }
};

// k = #{distinct list accuracies < min_acc}, from the bitmap with running popcounts.
template <class Img>
__device__ __forceinline__ uint32_t acc_rank(const Img &img, uint32_t bitmap_off, uint32_t acc_min,
                                             uint32_t x_max, uint32_t min_acc) {
  const uint32_t x = min(max(min_acc, acc_min) - acc_min, x_max);
  const uint32_t w = (x * 43691u) >> 20;                    // x / 24 for x < 2^16
  const uint32_t word = img.u32(bitmap_off + (w << 2));
  return (word >> 24) + __popc(word & ((1u << (x - w * ACC_WORD_BITS)) - 1u));
}

// Fast path, straight-line: five loads.  Returns the decision, INFAAS_INVALID, or PENDING
// when the query needs the slow path: nothing feasible, an SLO bucket with several values,
// or a task whose list has no index (those read 0xFF from T2 by construction).
template <class Img>
__device__ __forceinline__ uint32_t decide_fast(const Img &img, uint32_t n_tasks, uint32_t slo_off,
                                                uint32_t task, uint32_t slo, uint32_t min_acc) {
  const uint32_t t = min(task, n_tasks);
  const uint4 h = img.v4(t << 4);
  const uint32_t sh = (h.z >> 18) & 7u, bmin = h.w & 0x7FFFu;
  // r = #{distinct list latencies <= slo}: bucket record + one comparison
  const uint32_t b = (__float_as_uint(__uint2float_rz(slo)) >> 16) >> sh;
  const uint32_t j = min(max(b, bmin) - bmin, SLO_BUCKETS - 1u);
  const uint32_t lo = j ? __float2uint_ru(__uint_as_float((bmin + j) << (sh + 16u))) : 0u;
  const uint32_t rec = img.u32(slo_off + (((t << 8) + j) << 2));
  const uint32_t r = (rec >> 24) + ((slo - lo) >= (rec & 0x00FFFFFFu));
  const uint32_t k = acc_rank(img, h.y & 0x3FFFFu, h.x >> 18, h.w >> 15, min_acc);
  const uint32_t pos = img.u8((h.z & 0x3FFFFu) + r * (h.y >> 18) + k);
  const bool none = pos == 0xFFu;
  const uint32_t id = img.u32((h.x & 0x3FFFFu) + (none ? 0u : pos << 2));
  return none ? (((h.z >> 21) & HDR_FLAG_INVALID) ? INFAAS_INVALID : PENDING) : id;
}

// d = 10^4 * over_lat + slo * under_acc (64-bit).
__device__ __forceinline__ unsigned long long miss_distance(uint32_t pred, uint32_t acc, uint32_t slo,
                                                            uint32_t min_acc) {
  const uint32_t over = pred > slo ? pred - slo : 0u;
  const uint32_t under = min_acc > acc ? min_acc - acc : 0u;
  return (unsigned long long)over * 10000ull + (unsigned long long)slo * under;
}

// Slow path for a parked query (never an invalid one).
//   Indexed list: exact ranks (binary search over Pd), then T2.  If nothing is feasible the
//   nearest miss is the entry smallest in (d, position) -- position order is (cost,
//   pred_lat, -acc, id) order.  Entries that meet the SLO all miss the accuracy, the best
//   of them is the one with the highest accuracy (bestA); entries that meet the accuracy
//   all miss the SLO, the best being the one with the lowest latency (bestB); an entry
//   that misses both can only win with accuracy above bestA's, latency not above bestB's
//   and a latency overshoot that alone stays below the best distance so far, so the walk
//   in latency order stops early.
//   List without index: walk it in global memory, for a feasible entry, then for the distance.
template <class Img>
__device__ __forceinline__ uint32_t decide_slow(const Img &img, const DeviceCatalog &c, uint32_t task,
                                                uint32_t slo, uint32_t min_acc) {
  const uint4 h = img.v4(task << 4);
  unsigned long long best = ~0ull;
  uint32_t best_i = 0;
  if (!((h.z >> 21) & HDR_FLAG_NOT_INDEXED)) {
    const uint2 sl = img.v2(image_slow_offset(c.n_tasks) + (task << 3));
    const uint32_t F = sl.y & 0xFFu, Ks = (sl.y >> 8) & 0xFFu, Ka = sl.y >> 16;
    const uint32_t ids_off = h.x & 0x3FFFFu, pd_off = ids_off + (((F + 7u) >> 3) << 5);
    const AuxLayout AL = aux_layout(F, Ks, Ka);
    const uint32_t aux = sl.x;
    uint32_t lo = 0, hi = Ks;                              // r = #{Pd <= slo}
    while (lo < hi) {
      const uint32_t mid = (lo + hi) >> 1;
      if (img.u32(pd_off + (mid << 2)) <= slo) lo = mid + 1; else hi = mid;
    }
    const uint32_t r = lo;
    const uint32_t k = acc_rank(img, h.y & 0x3FFFFu, h.x >> 18, h.w >> 15, min_acc);
    const uint32_t pos = img.u8((h.z & 0x3FFFFu) + r * (h.y >> 18) + k);
    if (pos != 0xFFu) return img.u32(ids_off + (pos << 2));
    uint32_t acc_rank_floor = 0;          // candidates need accuracy rank >= this
    uint32_t lat_rank_cap = Ks;           // ... and latency rank < this
    if (r > 0) {                          // some entry meets the SLO (and misses the accuracy)
      const uint32_t pA = img.u8(aux + AL.bestA + r), ia = img.u8(aux + AL.idxA + pA);
      best = (unsigned long long)slo * (min_acc - img.u16(aux + AL.Ad + (ia << 1)));
      best_i = pA;
      acc_rank_floor = ia + 1u;
    }
    if (k < Ka) {                         // some entry meets the accuracy (and misses the SLO)
      const uint32_t pB = img.u8(aux + AL.bestB + k), ip = img.u8(aux + AL.idxP + pB);
      const unsigned long long d = (unsigned long long)(img.u32(pd_off + (ip << 2)) - slo) * 10000ull;
      if (d < best || (d == best && pB < best_i)) { best = d; best_i = pB; }
      lat_rank_cap = ip + 1u;
    }
    for (uint32_t o = img.u8(aux + AL.ordStart + r); o < F; ++o) {   // latency ranks >= r
      const uint32_t ip = img.u8(aux + AL.ordRank + o);
      if (ip >= lat_rank_cap) break;
      const unsigned long long over = (unsigned long long)(img.u32(pd_off + (ip << 2)) - slo) * 10000ull;
      if (over > best) break;             // later entries overshoot the SLO even more
      const uint32_t p = img.u8(aux + AL.order + o), ia = img.u8(aux + AL.idxA + p);
      if (ia >= acc_rank_floor && ia < k) {
        const unsigned long long d = over + (unsigned long long)slo * (min_acc - img.u16(aux + AL.Ad + (ia << 1)));
        if (d < best || (d == best && p < best_i)) { best = d; best_i = p; }
      }
    }
    return INFAAS_NO_FEASIBLE | img.u32(ids_off + (best_i << 2));
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
    const unsigned long long d = miss_distance((uint32_t)e, (uint32_t)(e >> 32), slo, min_acc);
    if (d < best) { best = d; best_i = i; }
  }
  return INFAAS_NO_FEASIBLE | __ldg(ids + best_i);
}

struct Queries {
  const uint16_t *__restrict__ task;
  const uint32_t *__restrict__ slo;
  const uint16_t *__restrict__ min_acc;
  uint32_t *__restrict__ decision;
};

// Resolve up to 32 parked queries, one per lane.  `rel` is the query's offset from `q0`.
template <class Img>
__device__ __forceinline__ void resolve_parked(const Img &img, const DeviceCatalog &c, const Queries &q,
                                               uint64_t q0, const uint32_t *park, uint32_t first,
                                               uint32_t count) {
  const uint32_t lane = threadIdx.x & 31;
  if (lane < count) {
    const uint64_t i = q0 + park[first + lane];
    q.decision[i] = decide_slow(img, c, q.task[i], q.slo[i], q.min_acc[i]);
  }
}

// Append the lanes with `pending` to the warp's park list (all lanes call this).
__device__ __forceinline__ void park_append(uint32_t *park, uint32_t &cnt, bool pending, uint32_t rel) {
  const unsigned m = __ballot_sync(0xFFFFFFFFu, pending);
  if (pending) park[cnt + __popc(m & ((1u << (threadIdx.x & 31)) - 1u))] = rel;
  cnt += __popc(m);
}

template <class Img>
__device__ __forceinline__ void select_body(const Img &img, const DeviceCatalog &c, const Queries &q,
                                            uint64_t n, uint64_t per_cta, uint32_t *park_all) {
  const uint32_t n_tasks = c.n_tasks;
  const uint32_t slo_off = image_slo_offset(n_tasks);
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t *park = park_all + warp * PARK_CAP;
  uint32_t parked = 0;
  const uint64_t q0 = (uint64_t)blockIdx.x * per_cta;
  const uint64_t q1 = min(n, q0 + per_cta);
  if (q0 >= q1) return;
  const uint64_t span = q1 - q0;                       // < 2^32 (checked by the launcher)
  const uint64_t full_tiles = span / WARP_TILE;

  // full tiles: 4 consecutive queries per lane, 128-bit loads, next tile prefetched
  uint64_t tile = warp;
  uint2 t4 = make_uint2(0, 0), a4 = make_uint2(0, 0);
  uint4 s4 = make_uint4(0, 0, 0, 0);
  if (tile < full_tiles) {
    const uint64_t i4 = (q0 + tile * WARP_TILE) / 4 + lane;
    t4 = __ldcs(reinterpret_cast<const uint2 *>(q.task) + i4);
    s4 = __ldcs(reinterpret_cast<const uint4 *>(q.slo) + i4);
    a4 = __ldcs(reinterpret_cast<const uint2 *>(q.min_acc) + i4);
  }
  for (; tile < full_tiles; tile += SELECT_WARPS) {
    const uint2 t = t4, a = a4;
    const uint4 s = s4;
    const uint64_t next = tile + SELECT_WARPS;
    if (next < full_tiles) {
      const uint64_t i4 = (q0 + next * WARP_TILE) / 4 + lane;
      t4 = __ldcs(reinterpret_cast<const uint2 *>(q.task) + i4);
      s4 = __ldcs(reinterpret_cast<const uint4 *>(q.slo) + i4);
      a4 = __ldcs(reinterpret_cast<const uint2 *>(q.min_acc) + i4);
    }
    uint4 d;
    d.x = decide_fast(img, n_tasks, slo_off, t.x & 0xFFFFu, s.x, a.x & 0xFFFFu);
    d.y = decide_fast(img, n_tasks, slo_off, t.x >> 16, s.y, a.x >> 16);
    d.z = decide_fast(img, n_tasks, slo_off, t.y & 0xFFFFu, s.z, a.y & 0xFFFFu);
    d.w = decide_fast(img, n_tasks, slo_off, t.y >> 16, s.w, a.y >> 16);
    const uint32_t rel = (uint32_t)(tile * WARP_TILE) + lane * 4u;
    uint32_t *out = q.decision + q0 + rel;
    const bool any_pending = d.x == PENDING || d.y == PENDING || d.z == PENDING || d.w == PENDING;
    if (!any_pending) {
      __stcs(reinterpret_cast<uint4 *>(out), d);
    } else {            // a parked slot is written later by another lane: leave it alone now
      if (d.x != PENDING) out[0] = d.x;
      if (d.y != PENDING) out[1] = d.y;
      if (d.z != PENDING) out[2] = d.z;
      if (d.w != PENDING) out[3] = d.w;
    }
    if (__any_sync(0xFFFFFFFFu, any_pending)) {
      park_append(park, parked, d.x == PENDING, rel);
      park_append(park, parked, d.y == PENDING, rel + 1);
      park_append(park, parked, d.z == PENDING, rel + 2);
      park_append(park, parked, d.w == PENDING, rel + 3);
      __syncwarp();
      while (parked >= 32) {
        parked -= 32;
        resolve_parked(img, c, q, q0, park, parked, 32);
      }
      __syncwarp();
    }
  }
  // ragged tail of the CTA's range (fewer than WARP_TILE queries): one warp, scalar accesses
  const uint64_t tail0 = full_tiles * WARP_TILE;
  if (tail0 < span && warp == (uint32_t)(full_tiles % SELECT_WARPS)) {
    for (uint32_t j = 0; j < WARP_TILE / 32; ++j) {
      const uint64_t rel = tail0 + j * 32u + lane;
      uint32_t d = 0;
      if (rel < span) {
        const uint64_t i = q0 + rel;
        d = decide_fast(img, n_tasks, slo_off, q.task[i], q.slo[i], q.min_acc[i]);
        if (d != PENDING) q.decision[i] = d;
      }
      park_append(park, parked, rel < span && d == PENDING, (uint32_t)rel);
    }
    __syncwarp();
    while (parked >= 32) {
      parked -= 32;
      resolve_parked(img, c, q, q0, park, parked, 32);
    }
  }
  __syncwarp();
  resolve_parked(img, c, q, q0, park, 0, parked);
}

__global__ void __launch_bounds__(SELECT_THREADS, 1)
select_kernel(DeviceCatalog c, uint32_t image_smem, Queries q, uint64_t n, uint64_t per_cta) {
  extern __shared__ __align__(128) unsigned char smem[];   // [park lists][staged image]
  __shared__ __align__(8) unsigned long long mbar;
  uint32_t *park = reinterpret_cast<uint32_t *>(smem);
  unsigned char *staged = smem + PARK_BYTES;
  const uint32_t bytes = c.image_hdr[0];
  if (bytes <= image_smem) {
    if (!stage_image(staged, c.image, bytes, &mbar)) {
      if (threadIdx.x == 0) atomicMax(c.err, (uint32_t)DEV_ERR_STAGE_TIMEOUT);
      return;
    }
    SharedImage img{smem_u32(staged)};
    select_body(img, c, q, n, per_cta, park);
  } else {
    // the image does not fit in shared memory: read it from global memory (L1/L2 resident)
    GlobalImage img{c.image};
    select_body(img, c, q, n, per_cta, park);
  }
}

}  // namespace

cudaError_t prepare_select_kernel() {
  return cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)SELECT_MAX_SMEM);
}

uint32_t select_image_smem(uint32_t image_smem) {
  if (image_smem + PARK_BYTES > SELECT_MAX_SMEM) image_smem = (SELECT_MAX_SMEM - PARK_BYTES) & ~15u;
  return image_smem;
}

cudaError_t launch_select(const DeviceCatalog &c, const uint16_t *d_task, const uint32_t *d_slo,
                          const uint16_t *d_min_acc, uint64_t n, uint32_t *d_decision,
                          int sm_count, uint32_t image_smem, cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  image_smem = select_image_smem(image_smem);
  // one CTA per SM; every CTA takes one contiguous range, a multiple of the warp tile
  uint64_t grid = (uint64_t)sm_count;
  const uint64_t tiles = (n + WARP_TILE - 1) / WARP_TILE;
  if (grid > tiles) grid = tiles;
  const uint64_t per_cta = (tiles + grid - 1) / grid * WARP_TILE;
  if (per_cta > 0xFFFFFFFFull) return cudaErrorInvalidValue;
  grid = (n + per_cta - 1) / per_cta;
  Queries q{d_task, d_slo, d_min_acc, d_decision};
  select_kernel<<<(uint32_t)grid, SELECT_THREADS, image_smem + PARK_BYTES, stream>>>(c, image_smem, q, n,
                                                                                     per_cta);
  return cudaGetLastError();
}

}  // namespace infaas
