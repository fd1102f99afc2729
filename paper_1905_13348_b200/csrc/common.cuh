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
// bucket's smallest slo); a bucket with two or more values is flagged and its record gives
// the range of Pd to compare against instead.  k comes from a bitmap over acc values with
// running popcounts (24 bitmap bits + 8 prefix bits per word), exact at one basis point.
//
// Image (what the selection kernel stages in shared memory), all parts 64-byte aligned:
//   hdr   u64[n_tasks]            per-task packed parameters (TaskHdr below)
//   slo   u32[n_tasks][SLO_BUCKETS]   SLO records: lb << 24 | delta, or flagged:
//                                     0xFF << 24 | lb << 8 | number of values in the bucket
//   var   per-task blocks back to back, each: ids u32[8*Fp8], Pd u32[8*Fp8],
//         acc bitmap u32[nbw], T2 u8[(Ks+1)*width], padded to 64 bytes
//
// Cold data (read from global memory by the slow path only), per task in its region, V =
// number of the task's variants:
//   keys u64[V] (F used)  pred_lat | acc_bp << 32 in scan order;  ids u32[V] (F used);
//   then, for an indexed list (Fi = min(V, INDEX_MAX_F)), what the nearest-miss search uses:
//   bestA u8[Fi+1]   bestA[r]: position of the highest accuracy among the r smallest latencies
//   bestB u8[Fi+1]   bestB[k]: position of the lowest latency among all but the k smallest accuracies
//   order u8[Fi]     positions sorted by latency rank;  ordStart u8[Fi+1]: first index of rank r
//   idxA u8[Fi], idxP u8[Fi]   accuracy / latency rank of each position
//   then, 64-byte aligned, the var block before it is packed into the image
// ---------------------------------------------------------------------------------------
constexpr uint32_t INDEX_MAX_F = 248;
constexpr uint32_t SLO_BUCKETS = 256;
constexpr uint32_t ACC_WORD_BITS = 24;
constexpr uint32_t MAX_ACC_WORDS = 420;          // covers 0..10000 bp at 24 per word
constexpr uint32_t SLO_FLAGGED = 0xFFu;
constexpr uint32_t VB_NOT_INDEXED = 0xFFEu;      // hdr.var_base value: list too long for the index
constexpr uint32_t VB_NO_VARIANTS = 0xFFFu;      // hdr.var_base value: the task has no variant

// hdr word 0: var_base (12 bits, units of 64 B from the start of the var section)
//             | acc_min4 << 12 (12 bits, units of 4 bp) | sh << 24 (3 bits) | Fp8 << 27 (5 bits)
// hdr word 1: bmin (15 bits) | nbw << 15 (9 bits) | width2 << 24 (7 bits, units of 2)
struct TaskHdr {
  uint32_t w0, w1;
};

inline __host__ __device__ uint32_t round_up_u32(uint32_t x, uint32_t a) { return (x + a - 1) / a * a; }

inline __host__ __device__ uint32_t image_slo_offset(uint32_t n_tasks) { return round_up_u32(8u * n_tasks, 64u); }
inline __host__ __device__ uint32_t image_var_offset(uint32_t n_tasks) {
  return image_slo_offset(n_tasks) + 4u * SLO_BUCKETS * n_tasks;
}

// Worst-case bytes of one task's var block and of its region (cold data + var block).
inline __host__ __device__ uint32_t var_capacity(uint32_t V) {
  const uint32_t F = V < INDEX_MAX_F ? V : INDEX_MAX_F;
  return round_up_u32(4u * MAX_ACC_WORDS + 8u * round_up_u32(F, 8) + (F + 1u) * (F + 2u), 64u);
}
struct ColdLayout {    // byte offsets inside a task's region
  uint32_t keys, ids, bestA, bestB, order, ordStart, idxA, idxP, var;
};
inline __host__ __device__ ColdLayout cold_layout(uint32_t V) {
  const uint32_t Fi = V < INDEX_MAX_F ? V : INDEX_MAX_F;
  ColdLayout L;
  L.keys = 0;
  L.ids = 8u * V;
  L.bestA = 12u * V;
  L.bestB = L.bestA + Fi + 1u;
  L.order = L.bestB + Fi + 1u;
  L.ordStart = L.order + Fi;
  L.idxA = L.ordStart + Fi + 1u;
  L.idxP = L.idxA + Fi;
  L.var = round_up_u32(L.idxP + Fi, 64u);
  return L;
}
inline __host__ __device__ uint32_t region_var_offset(uint32_t V) { return cold_layout(V).var; }
inline __host__ __device__ uint32_t region_capacity(uint32_t V) {
  return region_var_offset(V) + var_capacity(V);
}

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

  unsigned char *regions;    // per task: keys, Pd, then the var block before packing
  uint32_t *f_len;           // [n_tasks] list length F
  uint32_t *f_ks;            // [n_tasks] Ks | Ka << 16: distinct pred_lat / acc_bp values (0 if not indexed)
  uint32_t *f_var_bytes;     // [n_tasks] bytes of the task's var block (0 if not indexed)
  TaskHdr *f_hdr;            // [n_tasks] header words without var_base (filled in when packing)

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
// `image_smem`: bytes of dynamic shared memory reserved for the staged image (multiple of
// 16).  If the image is larger at run time the kernel reads it from global memory instead.
// Returns cudaErrorInvalidValue if n is too large for the launch geometry.
// Shared memory the launcher actually reserves for the image when asked for `image_smem`.
uint32_t select_image_smem(uint32_t image_smem);
cudaError_t launch_select(const DeviceCatalog &c, const uint16_t *d_task, const uint32_t *d_slo,
                          const uint16_t *d_min_acc, uint64_t n, uint32_t *d_decision,
                          int sm_count, uint32_t image_smem, cudaStream_t stream);

}  // namespace infaas
