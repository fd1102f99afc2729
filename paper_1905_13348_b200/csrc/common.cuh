// Shared declarations of the CUDA path: the device-side catalog layout and the launch
// functions the C ABI calls.  Nothing in this directory is used by, or uses, the CPU oracle.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "infaas.h"

namespace infaas {

// ---------------------------------------------------------------------------------------
// Device catalog.
//
// "Slot" order: variants bucketed by task, ascending id inside a task.  Task t owns slots
// task_off[t] .. task_off[t+1]-1.  All s_* arrays are indexed by slot.
//
// Scan list ("frontier") of a task: its non-dominated variants, sorted by
// (cost, pred_lat, 10000-acc, id).  Entry = one u64 key (pred_lat in bits 0..31, acc_bp in
// bits 32..47) plus the variant id.  Each task has a region of round_up(V_t, 4) entries in
// f_key / f_id at offset reg_off[t]; the first f_len[t] are valid.
//
// Blob: every task's scan list packed back to back, the image the selection kernel stages
// in shared memory with one bulk copy:
//     u32 table[2 * n_tasks_pad]   (start entry, length) per task
//     u64 keys [E_pad]             task t's keys at keys[start_t ...]
//     u32 ids  [E_pad]
// blob_hdr[0] = bytes of the whole image (multiple of 16), blob_hdr[1] = E_pad,
// blob_hdr[2] = longest list.  Offsets are fixed by n_tasks and E_pad only.
// ---------------------------------------------------------------------------------------
struct DeviceCatalog {
  uint32_t n_variants;
  uint32_t n_tasks;
  uint32_t n_tasks_pad;     // n_tasks rounded up to a multiple of 2 (table is 16-byte sized)
  uint32_t max_task_variants;
  uint32_t region_entries;  // sum over tasks of round_up(V_t, 4)

  const uint32_t *task_off;  // [n_tasks + 1]
  const uint32_t *reg_off;   // [n_tasks + 1]
  const uint32_t *s_lat;
  const uint16_t *s_batch;
  const uint16_t *s_acc;
  const uint32_t *s_cost;
  const uint32_t *s_id;
  uint32_t *s_queued;
  uint32_t *s_pred;
  unsigned long long *s_served;
  uint32_t *count_by_id;     // [n_variants], zero between windows

  unsigned long long *f_key;  // [region_entries]
  uint32_t *f_id;             // [region_entries]
  uint32_t *f_len;            // [n_tasks]

  unsigned char *blob;        // blob_capacity bytes, 16-byte aligned
  uint32_t blob_capacity;
  uint32_t *blob_hdr;         // [4]

  unsigned long long *counters;  // [3] feasible, no-feasible, invalid
  uint32_t *done_ctr;            // CTA arrival counter of the rebuild kernel
  uint32_t *err;                 // sticky device error word (0 = fine)
};

// Device error codes stored in DeviceCatalog::err.
enum : uint32_t {
  DEV_ERR_NONE = 0,
  DEV_ERR_STAGE_TIMEOUT = 1,  // the bulk copy into shared memory did not complete in time
  DEV_ERR_BLOB_OVERFLOW = 2,  // packed scan lists exceed the blob buffer (cannot happen by sizing)
};

inline __host__ __device__ uint32_t blob_table_bytes(uint32_t n_tasks_pad) {
  return n_tasks_pad * 8u;
}
inline __host__ __device__ uint32_t blob_total_bytes(uint32_t n_tasks_pad, uint32_t e_pad) {
  return n_tasks_pad * 8u + e_pad * 12u;
}

// Largest dynamic shared memory the selection kernel may be given (227 KB per CTA on
// sm_100, minus its static shared memory).
constexpr uint32_t SELECT_MAX_SMEM = 227u * 1024u - 256u;
constexpr uint32_t REBUILD_MAX_SMEM = INFAAS_MAX_TASK_VARIANTS * 12u;

// Once per device, with that device current: raise the kernels' shared-memory limits.
cudaError_t prepare_select_kernel();
cudaError_t prepare_rebuild_kernel();

// Launchers (host).  All are asynchronous on `stream` and allocate nothing.
cudaError_t launch_rebuild(const DeviceCatalog &c, bool advance_queues, uint32_t window_us,
                           cudaStream_t stream);
cudaError_t launch_tally(const DeviceCatalog &c, const uint32_t *d_decision, uint64_t n,
                         cudaStream_t stream);
// `smem_bytes`: dynamic shared memory for the staged image (multiple of 16).  If the image
// is larger at run time the kernel scans it in global memory instead.
cudaError_t launch_select(const DeviceCatalog &c, const uint16_t *d_task, const uint32_t *d_slo,
                          const uint16_t *d_min_acc, uint64_t n, uint32_t *d_decision,
                          int sm_count, uint32_t smem_bytes, cudaStream_t stream);

}  // namespace infaas
