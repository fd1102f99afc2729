// Shared declarations of the CUDA path: the device-side catalog layout, the packed image
// the selection kernel reads, and the launch functions the C ABI calls.  Nothing in this
// directory is used by, or uses, the CPU oracle.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "infaas.h"

namespace infaas {

// ---------------------------------------------------------------------------------------
// Scan list of a task: its non-dominated variants sorted by (cost, pred_lat, 10000-acc, id).
// Position p in that order is what selection returns the smallest feasible of.
//
// For a list of F <= INDEX_MAX_F entries the rebuild kernel derives an exact index:
//   Pd[0..Ks)  distinct pred_lat values ascending,  Ad[0..Ka)  distinct acc_bp ascending,
//   r(slo) = #{Pd <= slo},  k(min_acc) = #{Ad < min_acc},
//   T2[r][k] = first position whose pred_lat is among the r smallest values and whose
//              acc_bp is not among the k smallest values (0xFF: none) -- the answer.
// r comes from a table of SLO_BUCKETS records indexed by a monotone bucket of slo (top bits
// of slo converted to float, shifted by `sh`, relative to `bmin`); a record holds the rank
// below the bucket and the one distinct value inside it (as a 24-bit offset from the
// bucket's smallest slo).  A bucket holding two or more values sends the query to two
// extra rows of T2 that contain only 0xFF, i.e. to the exact slow path.  k comes from a
// bitmap over acc values with running popcounts (24 bitmap bits + 8 prefix bits per word),
// exact at one basis point.
//
// Image (what the selection kernel stages in shared memory), all parts 64-byte aligned:
//   hdr    uint4[n_tasks + 1]   fast-path parameters (below); entry n_tasks serves queries
//                               whose task is out of range
//   slow   uint2[n_tasks + 1]   slow-path parameters: aux offset, F | Ks<<8 | Ka<<16
//   slo    u32[n_tasks + 1][SLO_BUCKETS]   SLO records: lb << 24 | delta
//   dummy  64 bytes of 0x00, 64 bytes of 0xFF   (what tasks without an index point at)
//   var    per-task blocks back to back, each:
//          ids u32[8*Fp8], Pd u32[8*Fp8], acc bitmap u32[nbw], T2 u8[(Ks+3)*width],
//          aux (what the nearest-miss search reads, see AuxLayout), padded to 64 bytes
//
// hdr words (offsets are bytes from the start of the image, 18 bits):
//   x = ids_off | acc_min << 18            y = bitmap_off | width << 18
//   z = t2_off | sh << 18 | flags << 21    w = bmin | x_max << 15     (x_max = 24*nbw - 1)
//
// Per task in its region (global memory): keys u64[V] (pred_lat | acc_bp << 32, scan
// order, F used), ids u32[V]; then, 64-byte aligned, the var block before it is packed.
// ---------------------------------------------------------------------------------------
constexpr uint32_t INDEX_MAX_F = 248;
constexpr uint32_t SLO_BUCKETS = 256;
constexpr uint32_t ACC_WORD_BITS = 24;
constexpr uint32_t MAX_ACC_WORDS = 420;          // covers 0..10000 bp at 24 per word
constexpr uint32_t IMAGE_OFFSET_LIMIT = 1u << 18;
constexpr uint32_t HDR_FLAG_INVALID = 1u;        // no variant (or task out of range): answer INVALID
constexpr uint32_t HDR_FLAG_NOT_INDEXED = 2u;    // list without index: the slow path walks it

inline __host__ __device__ uint32_t round_up_u32(uint32_t x, uint32_t a) { return (x + a - 1) / a * a; }

inline __host__ __device__ uint32_t image_slow_offset(uint32_t n_tasks) { return round_up_u32(16u * (n_tasks + 1u), 64u); }
inline __host__ __device__ uint32_t image_slo_offset(uint32_t n_tasks) {
  return image_slow_offset(n_tasks) + round_up_u32(8u * (n_tasks + 1u), 64u);
}
inline __host__ __device__ uint32_t image_dummy_offset(uint32_t n_tasks) {
  return image_slo_offset(n_tasks) + 4u * SLO_BUCKETS * (n_tasks + 1u);
}
inline __host__ __device__ uint32_t image_var_offset(uint32_t n_tasks) { return image_dummy_offset(n_tasks) + 128u; }

// Byte offsets inside the aux part of a var block, for a list of F entries with Ks / Ka
// distinct latencies / accuracies.
//   bestA[r], r in 0..Ks: position of the highest accuracy among the r smallest latencies
//   bestB[k], k in 0..Ka: position of the lowest latency among all but the k smallest accuracies
//   order[o]: positions sorted by latency rank; ordRank[o]: that rank; ordStart[r]: first o of rank r
//   idxA[p], idxP[p]: accuracy / latency rank of position p;  Ad u16[Ka]: distinct accuracies
struct AuxLayout {
  uint32_t bestA, bestB, order, ordRank, ordStart, idxA, idxP, Ad, bytes;
};
inline __host__ __device__ AuxLayout aux_layout(uint32_t F, uint32_t Ks, uint32_t Ka) {
  AuxLayout L;
  L.bestA = 0;
  L.bestB = L.bestA + Ks + 1u;
  L.order = L.bestB + Ka + 1u;
  L.ordRank = L.order + F;
  L.ordStart = L.ordRank + F;
  L.idxA = L.ordStart + Ks + 1u;
  L.idxP = L.idxA + F;
  L.Ad = (L.idxP + F + 1u) & ~1u;
  L.bytes = L.Ad + 2u * Ka;
  return L;
}

// Worst-case bytes of one task's var block and of its region.
inline __host__ __device__ uint32_t var_capacity(uint32_t V) {
  const uint32_t F = V < INDEX_MAX_F ? V : INDEX_MAX_F;
  return round_up_u32(8u * round_up_u32(F, 8) + 4u * MAX_ACC_WORDS + (F + 3u) * (F + 2u) +
                          aux_layout(F, F, F).bytes, 64u);
}
inline __host__ __device__ uint32_t region_var_offset(uint32_t V) { return round_up_u32(12u * V, 64u); }
inline __host__ __device__ uint32_t region_capacity(uint32_t V) { return region_var_offset(V) + var_capacity(V); }

// ---------------------------------------------------------------------------------------
// Device catalog.  "Slot" order: variants bucketed by task, ascending id inside a task;
// task t owns slots task_off[t] .. task_off[t+1]-1 and all s_* arrays are indexed by slot.
// ---------------------------------------------------------------------------------------
struct DeviceCatalog {
  uint32_t n_variants;
  uint32_t n_tasks;
  uint32_t max_task_variants;

  const uint32_t *task_off;  // [n_tasks + 1]
  const uint32_t *reg_off;   // [n_tasks + 1] byte offset of each task's region
  const uint32_t *s_lat;
  const uint16_t *s_batch;
  const uint16_t *s_acc;
  const uint32_t *s_cost;
  const uint32_t *s_id;
  uint32_t *s_queued;
  uint32_t *s_pred;
  unsigned long long *s_served;
  uint32_t *count_by_id;     // [n_variants], zero between windows

  unsigned char *regions;    // per task: keys, ids, then the var block before packing
  uint32_t *f_len;           // [n_tasks] list length F
  uint32_t *f_var_bytes;     // [n_tasks] bytes of the task's var block (0 if not indexed)
  uint4 *f_hdr;              // [n_tasks] hdr words with offsets relative to the var block
  uint2 *f_slow;             // [n_tasks] slow words, aux offset relative to the var block

  unsigned char *image;      // packed image, image_capacity bytes, 256-byte aligned
  uint32_t image_capacity;
  uint32_t *image_hdr;       // [4]: bytes, longest list, total entries, tasks not indexed

  unsigned long long *counters;  // [3] feasible, no-feasible, invalid
  uint32_t *done_ctr;            // CTA arrival counter of the rebuild kernel
  uint32_t *err;                 // sticky device error word (0 = fine)
};

// Device error codes stored in DeviceCatalog::err.
enum : uint32_t {
  DEV_ERR_NONE = 0,
  DEV_ERR_STAGE_TIMEOUT = 1,   // the bulk copy into shared memory did not complete in time
  DEV_ERR_IMAGE_OVERFLOW = 2,  // packed image exceeds its buffer (cannot happen by sizing)
};

// Largest dynamic shared memory the selection kernel may be given (227 KB per CTA on
// sm_100, minus its static shared memory).
constexpr uint32_t SELECT_MAX_SMEM = 227u * 1024u - 256u;
// Sort buffers of the rebuild kernel: 13 bytes per padded entry.
constexpr uint32_t REBUILD_MAX_SMEM = INFAAS_MAX_TASK_VARIANTS * 13u;

// Once per device, with that device current: raise the kernels' shared-memory limits.
cudaError_t prepare_select_kernel();
cudaError_t prepare_rebuild_kernel();

// Launchers (host).  All are asynchronous on `stream` and allocate nothing.
cudaError_t launch_rebuild(const DeviceCatalog &c, bool advance_queues, uint32_t window_us,
                           cudaStream_t stream);
cudaError_t launch_tally(const DeviceCatalog &c, const uint32_t *d_decision, uint64_t n,
                         cudaStream_t stream);
// Shared memory the launcher actually reserves for the image when asked for `image_smem`.
uint32_t select_image_smem(uint32_t image_smem);
// `image_smem`: bytes of dynamic shared memory reserved for the staged image (multiple of
// 16).  If the image is larger at run time the kernel reads it from global memory instead.
// Returns cudaErrorInvalidValue if n is too large for the launch geometry.
cudaError_t launch_select(const DeviceCatalog &c, const uint16_t *d_task, const uint32_t *d_slo,
                          const uint16_t *d_min_acc, uint64_t n, uint32_t *d_decision,
                          int sm_count, uint32_t image_smem, cudaStream_t stream);

}  // namespace infaas
