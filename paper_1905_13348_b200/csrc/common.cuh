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
// A state-aware catalog has two lists per task, one after the other: the Active variants in
// the order above, then the Inactive ones with pred_lat + loading latency (saturating) in
// place of both cost and pred_lat; each list is pruned on its own, variants in other states
// are in neither.  "First feasible position, else the smallest distance at the lowest
// position" over the two lists in this order is the state-aware answer, and that is all the
// index below knows about order, so the two lists are indexed as one.
//
// A list is cut into segments of at most INDEX_MAX_F consecutive positions (almost always
// one).  The selection kernel's fast path looks at the first segment only; if that holds
// nothing feasible the slow path goes through the others in order.  For a segment of F
// entries the rebuild kernel derives an exact index:
//   Pd[0..Ks)  distinct pred_lat values ascending,  Ad[0..Ka)  distinct acc_bp ascending,
//   r(slo) = #{Pd <= slo},  k(min_acc) = #{Ad < min_acc},
//   T2[r][k] = first position whose pred_lat is among the r smallest values and whose
//              acc_bp is not among the k smallest values, or F if there is none.
//
// r comes from one record of a table of SLO_BUCKETS records per task.  The bucket of an
// SLO is  j = clamp((bits(slo) >> S) - bmin, 0, 255)  with bits(x) = the IEEE-754 pattern
// of x converted to float toward zero (a monotone, roughly logarithmic code) and one S = 16..23
// and bmin for the whole catalog.  A record is  R << 24 | C  and
// r = (record + (slo & 0xFFFFFF)) >> 24:
//   - no distinct latency inside the bucket: R = the rank there, C = 0 (never carries);
//   - one latency `thr` inside it, and all SLOs of the bucket agree in their top byte:
//     R = rank below, C = 0xFFFFFF - ((thr - 1) & 0xFFFFFF), so the add carries into R
//     exactly when slo >= thr;
//   - otherwise R = Ks + 1, C = 0: row Ks + 1 of T2 holds only F, which sends the query to
//     the exact slow path.
// The buckets run from the smallest profiled latency of the catalog (a predicted latency is
// never below it) up to the largest SLO any batch has asked for so far (kept as a bit mask,
// at least SLO_CAP_FLOOR_US); larger latencies share bucket 255.  The rebuild kernel derives
// S and bmin from these two and publishes them beside the image size.
// k comes from a bitmap over accuracy values with running popcounts (24 bitmap bits and an
// 8-bit prefix count per word), exact at one basis point.  Every bitmap covers the same
// window of accuracies, that of the whole catalog (fixed at load: acc_lo, a multiple of 24,
// and nbw words), so the word an accuracy falls into does not depend on the task.
//
// Image (what the selection kernel stages in shared memory):
//   dummy  64 bytes (what tasks without an index point at: every query of theirs reads
//          "none" and goes to the slow path)
//   hdr    (n_tasks + 1) u32, one per task: t2_off | (Ka + 1) << 24; entry n_tasks serves
//          queries whose task is out of range; padded to 128 bytes
//   rec    (n_tasks + 1) x SLO_BUCKETS u32 records, REC_STRIDE bytes apart
//   bitmap (n_tasks + 1) x nbw u32: the accuracy bitmaps of the tasks' first segments,
//          bitmap_stride(nbw) bytes apart
//   var    per-segment blocks, each 16-byte aligned:
//          ids   u32[F + 1] in REVERSE order: ids[p] sits at t2_off - 4 - 4p, and the slot
//                of p = F holds PENDING -- the fast path needs no compare for "none"
//          T2    u8[(Ks + 2) * (Ka + 1)]  at t2_off (a multiple of 4)
//          bitmap u32[nbw]  (further segments only)
//          slow-path tables (SlowLayout below)
//
// Per task in global memory (`regions`): keys u64[V] (pred_lat | acc_bp << 32, scan order,
// F used; for Inactive entries the latency includes the loading latency) and ids u32[V], for
// lists without an index and for inspection; then local u16[V], the entries' indices inside
// the task, which the next rebuild uses as its first filter.
// ---------------------------------------------------------------------------------------
constexpr uint32_t INDEX_MAX_F = 248;
constexpr uint32_t SLO_BUCKETS = 256;
constexpr uint32_t ACC_WORD_BITS = 24;
constexpr uint32_t MAX_ACC_WORDS = 420;          // accuracies 0 .. 10000 need at most 417 + 1 words
constexpr uint32_t IMAGE_T2_LIMIT = 1u << 24;    // t2_off is a 24-bit field
constexpr uint32_t SLO_CAP_FLOOR_US = (1u << 20) - 1u;  // the buckets cover latencies at least up to here
constexpr uint32_t PENDING = 0xFFFFFFFEu;        // never a valid decision (ids stop at 2^31-2)

constexpr uint32_t TASK_FLAG_INVALID = 1u;       // no variant: answer INFAAS_INVALID
constexpr uint32_t TASK_FLAG_NOT_INDEXED = 2u;   // list without index: the slow path walks it

inline __host__ __device__ uint32_t round_up_u32(uint32_t x, uint32_t a) { return (x + a - 1) / a * a; }

// A task's records and its bitmap start an odd number of words after the previous task's, so
// that the tasks' hot entries (the same buckets, the lowest bitmap word) fall into different
// shared-memory banks.
constexpr uint32_t REC_STRIDE = 4u * (SLO_BUCKETS + 1u);   // bytes from one task's records to the next's
inline __host__ __device__ uint32_t bitmap_stride(uint32_t nbw) { return 4u * (nbw | 1u); }   // same, bitmaps
constexpr uint32_t IMAGE_DUMMY_BYTES = 64u;               // the dummy block opens the image
constexpr uint32_t IMAGE_HDR_OFFSET = IMAGE_DUMMY_BYTES;  // the task words follow it
inline __host__ __device__ uint32_t image_rec_offset(uint32_t n_tasks) {
  return round_up_u32(IMAGE_HDR_OFFSET + 4u * (n_tasks + 1u), 128u);
}
inline __host__ __device__ uint32_t image_bitmap_offset(uint32_t n_tasks) {
  return image_rec_offset(n_tasks) + REC_STRIDE * (n_tasks + 1u);
}
inline __host__ __device__ uint32_t image_var_offset(uint32_t n_tasks, uint32_t nbw) {
  return round_up_u32(image_bitmap_offset(n_tasks) + bitmap_stride(nbw) * (n_tasks + 1u), 64u);
}
// The task word of a task without index (and of entry n_tasks): T2 is the one zero byte at
// offset 16 of the dummy block with row width 0, the id slot of position 0 below it holds
// PENDING.  The dummy block sits at the very start of the image, where the task word's 24-bit
// offset reaches it however large the fixed tables are.
constexpr uint32_t DUMMY_HEADER = 16u;

// Byte offsets of the slow-path tables inside a segment's block, relative to their start
// (8-byte aligned), for a list of F entries with Ks / Ka distinct latencies / accuracies.
//   walk[o]   uint2 (pred_lat, acc | position << 16): the "stair" entries -- those no other
//             entry beats in both latency and accuracy -- in ascending latency (Fs <= F of
//             them, all with different latencies; space for F)
//   bestB[k]  uint2 (pred_lat, position) of the lowest-latency entry among those whose
//             accuracy rank is >= k (first position among equals); position 0xFF if none
//   Pd[i]     u32 distinct latencies
//   bestA[r]  u32 acc | position << 16 of the highest-accuracy entry among those whose
//             latency rank is < r (first position among equals); position 0xFF if none
//   ordStart[r] u8 first walk index whose latency rank is >= r
struct SlowLayout {
  uint32_t walk, bestB, Pd, bestA, ordStart, bytes;
};
inline __host__ __device__ SlowLayout slow_layout(uint32_t F, uint32_t Ks, uint32_t Ka) {
  SlowLayout L;
  L.walk = 0;
  L.bestB = L.walk + 8u * F;
  L.Pd = L.bestB + 8u * (Ka + 1u);
  L.bestA = L.Pd + 4u * Ks;
  L.ordStart = L.bestA + 4u * (Ks + 1u);
  L.bytes = round_up_u32(L.ordStart + Ks + 1u, 8u);
  return L;
}

// Offsets inside a segment's block and its size; `nbw` = 0 for a task's first segment (its
// bitmap lives in the fixed part of the image).
struct BlockLayout {
  uint32_t t2, bitmap, slow, bytes;   // ids start at 0; t2 = 4 (F + 1)
};
inline __host__ __device__ BlockLayout block_layout(uint32_t F, uint32_t Ks, uint32_t Ka, uint32_t nbw) {
  BlockLayout B;
  B.t2 = 4u * (F + 1u);
  B.bitmap = round_up_u32(B.t2 + (Ks + 2u) * (Ka + 1u), 4u);
  B.slow = round_up_u32(B.bitmap + 4u * nbw, 8u);
  B.bytes = round_up_u32(B.slow + slow_layout(F, Ks, Ka).bytes, 16u);
  return B;
}
// Worst-case bytes of one segment's block.
inline __host__ __device__ uint32_t block_capacity(uint32_t V, uint32_t nbw) {
  const uint32_t F = V < INDEX_MAX_F ? V : INDEX_MAX_F;
  return block_layout(F, F, F, nbw).bytes;
}
inline __host__ __device__ uint32_t region_capacity(uint32_t V) { return round_up_u32(14u * V, 64u); }

// Slow-path parameters of a list segment (one uint4 each, global memory; a task's first
// segment at index task, further segments at n_tasks + their index).
//   x = image offset of the slow tables   y = F | Ks << 8 | Ka << 16   z = flags
//   w = Fs | (1 + index of the task's next segment, 0 if none) << 8
// Header of a further segment (xhdr, global memory):
//   x = t2_off   y = Ka + 1   z = image offset of its bitmap   w = 0
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
  uint32_t stateful;         // 1: states and loading latencies below take part (else all Active)
  unsigned char *s_state;    // INFAAS_STATE_* per slot
  const uint32_t *s_load_lat;  // loading latency per slot, microseconds

  unsigned char *regions;    // per task: keys u64[V], ids u32[V] (scan order)
  uint32_t *f_len;           // [n_tasks] list length F
  uint4 *slow;               // [n_tasks + n_extra] slow-path parameters of the segments
  const uint32_t *seg_base;  // [n_tasks + 1] index of each task's first further segment
  uint4 *xhdr;               // [n_extra] headers of the further segments (first segments: in the image)

  unsigned char *image;      // packed image, image_capacity bytes, 256-byte aligned
  uint32_t image_capacity;
  uint32_t *image_hdr;       // published by the rebuild kernel: [0] bytes of the image, [1] the bucket
                             // scale 2^-S and [2] -bmin, both as float patterns
  uint32_t acc_lo, nbw;      // accuracy window of every bitmap: acc_lo (multiple of 24) .. acc_lo + 24 nbw - 1
  uint32_t lat_code_lo;      // bits(smallest profiled latency) >> 16: where the SLO buckets start

  unsigned long long *counters;  // [3] feasible, no-feasible, invalid
  unsigned long long *alloc_ctr; // rebuild kernel: block cursor (low 32 bits) | CTAs done allocating << 32;
                                 // zero between kernels
  uint32_t *err;                 // sticky device error word (0 = fine)
  uint32_t *slo_seen;            // OR of all SLOs the selection kernel has read
};

// Device error codes stored in DeviceCatalog::err.
enum : uint32_t {
  DEV_ERR_NONE = 0,
  DEV_ERR_STAGE_TIMEOUT = 1,   // the bulk copy into shared memory did not complete in time
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
                         int sm_count, cudaStream_t stream);
// Shared memory the launcher actually reserves for the image when asked for `image_smem`.
uint32_t select_image_smem(uint32_t image_smem);
// `image_smem`: bytes of dynamic shared memory reserved for the staged image (multiple of
// 16).  If the image is larger at run time the kernel reads it from global memory instead.
// `tally`: the kernel also adds the decisions to the pending per-variant counts and the
// catalog's counters (what launch_tally would do with them).
// Returns cudaErrorInvalidValue if n is too large for the launch geometry.
cudaError_t launch_select(const DeviceCatalog &c, const uint16_t *d_task, const uint32_t *d_slo,
                          const uint16_t *d_min_acc, uint64_t n, uint32_t *d_decision,
                          int sm_count, uint32_t image_smem, bool tally, cudaStream_t stream);
// Batches below this size are tallied by the selection kernel itself in infaas_select_update.
constexpr uint64_t FUSED_TALLY_MAX_N = 1u << 18;

// Scaling-up step of the Model-Autoscaler for every task, from the pending per-variant
// counts; s_inst / s_arch / s_qps (floor(10^9 * batch / lat_us)) are per slot, task_slo per
// task; outputs have n_tasks entries.
cudaError_t launch_autoscale(const DeviceCatalog &c, const uint32_t *s_inst, const uint16_t *s_arch,
                             const unsigned long long *s_qps, const uint32_t *task_slo, uint32_t window_us, uint32_t slack_pct,
                             uint32_t lambda_milli, uint32_t *d_variant, uint32_t *d_delta,
                             cudaStream_t stream);

// Worker choice.  Build: one worker per variant from the instance table {variant, worker, load}
// and the worker table {hardware code, utilisation} (device arrays); best_inst [n_variants] and
// best_hw [256] are scratch.  Assign: worker[q] = worker_of[decision[q]] for decisions below
// n_variants, INFAAS_INVALID otherwise.
cudaError_t launch_workers_build(uint32_t n_variants, const unsigned char *hw_by_id,
                                 const uint32_t *inst_variant, const uint32_t *inst_worker,
                                 const uint32_t *inst_load, uint32_t n_inst, const unsigned char *worker_hw,
                                 const uint32_t *worker_util, uint32_t n_workers,
                                 unsigned long long *best_inst, unsigned long long *best_hw,
                                 uint32_t *worker_of, cudaStream_t stream);
cudaError_t launch_assign_workers(const uint32_t *d_decision, uint64_t n, uint32_t n_variants,
                                  const uint32_t *worker_of, uint32_t *d_worker, int sm_count,
                                  cudaStream_t stream);

// Integer-pipe probe: two CTAs per SM run `iters` steps of independent add / xor / compare /
// conditional-add chains; *lane_ops receives the number of lane-operations the launch executes.
cudaError_t launch_intpipe_probe(uint32_t iters, uint32_t seed, uint32_t *d_sink, int sm_count,
                                 unsigned long long *lane_ops, cudaStream_t stream);

// Remembers a CUDA error's text for infaas_last_cuda_error() (calling thread) and clears the
// runtime's error state; returns INFAAS_E_CUDA.
int record_cuda_error(cudaError_t e);

}  // namespace infaas
