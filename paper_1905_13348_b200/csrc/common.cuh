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
// Task block (one per task, 16-byte aligned, self-contained).  For a list of F entries:
//     keys   u64[F]   pred_lat (bits 0..31) | acc_bp (bits 32..47), scan order
//     ids    u32[F]   variant ids, scan order
//   and, if F <= MASK_MAX_F (the "indexed" form, nw = ceil(F/64) mask words):
//     thr    u32[F]   pred_lat ascending
//     accs   u16[F]   acc_bp ascending                      (padded to 4 bytes)
//     startL u8[260]  per SLO bucket: lower bound of #{thr <= slo}   (257 used)
//     startA u8[128]  per accuracy bucket: lower bound of #{accs < min_acc}
//     ML     u64[(F+1)*nw]   ML[r] = positions whose pred_lat is among the r smallest
//     MA     u64[(F+1)*nw]   MA[k] = positions whose acc_bp is NOT among the k smallest
//   A query with r = #{thr <= slo} and k = #{accs < min_acc} is met exactly by the
//   positions in ML[r] & MA[k]; the answer is the lowest set bit.
//   SLO bucket of s: 0 for s = 0, else 1 + (eighth-octave index of s) -- the top 11 bits
//   of s converted to float (round toward zero), minus 1015.
//   Accuracy bucket of m: min(127, max(0, m - acc_base) >> acc_shift).
//
// Image: TaskDesc[n_tasks] followed by the blocks back to back; this is what the
// selection kernel stages in shared memory.  All offsets in a TaskDesc are bytes from the
// start of the image.
// ---------------------------------------------------------------------------------------
constexpr uint32_t MASK_MAX_F = 256;
constexpr uint32_t SLO_BUCKETS = 257;
constexpr uint32_t SLO_BUCKET_BYTES = 260;
constexpr uint32_t ACC_BUCKETS = 128;
constexpr uint32_t SLO_BUCKET_BIAS = 1015;   // (127 << 3) - 1: float exponent of 1.0, three mantissa bits

struct __align__(16) TaskDesc {   // 32 bytes
  uint32_t off_masks;   // ML; MA follows (F+1)*nw words later
  uint32_t f_nw;        // F | nw << 16 ; nw == 0: not indexed (linear scan)
  uint32_t acc_meta;    // acc_base | acc_shift << 16
  uint32_t off_keys;
  uint32_t off_thr;
  uint32_t off_ids;
  uint32_t off_accs;
  uint32_t off_start;   // startL; startA is SLO_BUCKET_BYTES further
};

struct BlockLayout {    // byte offsets inside a task block
  uint32_t keys, ids, thr, accs, start, masks, bytes, nw;
};

inline __host__ __device__ BlockLayout block_layout(uint32_t F) {
  BlockLayout L;
  L.nw = (F > 0 && F <= MASK_MAX_F) ? (F + 63u) / 64u : 0u;
  L.keys = 0;
  L.ids = 8u * F;
  uint32_t end = 12u * F;
  L.thr = L.accs = L.start = L.masks = end;
  if (L.nw) {
    L.thr = end;
    L.accs = L.thr + 4u * F;
    L.start = L.accs + ((2u * F + 3u) & ~3u);
    L.masks = (L.start + SLO_BUCKET_BYTES + ACC_BUCKETS + 7u) & ~7u;
    end = L.masks + 16u * (F + 1u) * L.nw;
  }
  L.bytes = (end + 15u) & ~15u;
  return L;
}

// Largest block a task with V variants can need (every variant non-dominated, or the
// longest indexed list, whichever is larger).
inline __host__ __device__ uint32_t block_capacity(uint32_t V) {
  uint32_t a = block_layout(V).bytes;
  uint32_t b = block_layout(V < MASK_MAX_F ? V : MASK_MAX_F).bytes;
  return a > b ? a : b;
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
  const uint32_t *reg_off;   // [n_tasks + 1] byte offset of each task's block region
  const uint32_t *s_lat;
  const uint16_t *s_batch;
  const uint16_t *s_acc;
  const uint32_t *s_cost;
  const uint32_t *s_id;
  uint32_t *s_queued;
  uint32_t *s_pred;
  unsigned long long *s_served;
  uint32_t *count_by_id;     // [n_variants], zero between windows

  unsigned char *regions;    // task blocks at their worst-case offsets (16-byte aligned)
  uint32_t *f_len;           // [n_tasks] list length F
  uint32_t *f_meta;          // [n_tasks] acc_base | acc_shift << 16

  unsigned char *image;      // packed image, image_capacity bytes, 16-byte aligned
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
cudaError_t launch_select(const DeviceCatalog &c, const uint16_t *d_task, const uint32_t *d_slo,
                          const uint16_t *d_min_acc, uint64_t n, uint32_t *d_decision,
                          int sm_count, uint32_t image_smem, cudaStream_t stream);

}  // namespace infaas
