// C ABI of the library (declared in include/infaas.h): handle management, validation,
// the host side of the catalog packer, and the calls that launch the kernels.
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "common.cuh"

using infaas::DeviceCatalog;

struct infaas_catalog {
  int device = 0;
  int sm_count = 0;
  DeviceCatalog d{};
  void *arena = nullptr;                 // one device allocation holds every array
  std::vector<uint32_t> slot_of_id;      // host copy, for get_state
  std::vector<uint32_t> task_off, reg_off;
  uint32_t select_smem = 0;              // shared memory reserved for the staged image
  uint32_t worst_image_bytes = 0;        // image size if every block had its largest size
  uint32_t *s_inst = nullptr;            // running instances per slot (Model-Autoscaler)
  uint16_t *s_arch = nullptr;            // architecture code per slot
  unsigned long long *s_qps = nullptr;   // profiled saturation throughput per slot, milli-queries/s
  uint32_t *task_slo = nullptr;          // SLO per task
  bool autoscale_ready = false;
  unsigned char *hw_by_id = nullptr;     // hardware code per variant id (worker choice)
  uint32_t *worker_of = nullptr;         // worker per variant id
  unsigned long long *best_inst = nullptr, *best_hw = nullptr;   // scratch of the table build
  bool workers_ready = false;
};

namespace {

thread_local std::string g_cuda_error;

int cuda_fail(cudaError_t e) {
  g_cuda_error = std::string(cudaGetErrorName(e)) + ": " + cudaGetErrorString(e);
  (void)cudaGetLastError();   // clear the sticky-free error state
  return INFAAS_E_CUDA;
}

// Multiprocessors of a device, asked once per device.
int sm_count_of(int device) {
  static int cached[64] = {};
  if (device < 0 || device >= 64) return 0;
  if (!cached[device]) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return 0;
    cached[device] = n;
  }
  return cached[device];
}

#define CUDA_TRY(expr)                         \
  do {                                         \
    cudaError_t e__ = (expr);                  \
    if (e__ != cudaSuccess) return cuda_fail(e__); \
  } while (0)

// Makes the catalog's device current for the scope of one call.
struct DeviceScope {
  int prev = -1;
  bool switched = false;
  cudaError_t status = cudaSuccess;
  explicit DeviceScope(int dev) {
    status = cudaGetDevice(&prev);
    if (status == cudaSuccess && prev != dev) {
      status = cudaSetDevice(dev);
      switched = status == cudaSuccess;
    }
  }
  ~DeviceScope() {
    if (switched) (void)cudaSetDevice(prev);
  }
};

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// IEEE-754 single-precision pattern of x (> 0) converted toward zero, as the kernels compute it.
inline uint32_t float_bits_rz(uint32_t x) {
  uint32_t e = 31;
  while (!(x >> e)) --e;
  const uint32_t mant = (uint32_t)(((uint64_t)x << (31 - e)) >> 8) & 0x7FFFFFu;
  return ((e + 127u) << 23) | mant;
}

// Re-reads the image size from the device and decides how much shared memory the selection
// kernel asks for: all of it while the image fits (it may grow or shrink between two such
// refreshes without a change of plan), none for the image if it does not -- the kernel
// then reads it from global memory and the space is worth more as L1 cache.
int refresh_select_plan(infaas_catalog *c, cudaStream_t stream) {
  uint32_t hdr[1] = {0};
  CUDA_TRY(cudaMemcpyAsync(hdr, c->d.image_hdr, sizeof(hdr), cudaMemcpyDeviceToHost, stream));
  CUDA_TRY(cudaStreamSynchronize(stream));
  const uint32_t room = infaas::select_image_smem(infaas::SELECT_MAX_SMEM);
  c->select_smem = hdr[0] <= room ? room : 0u;
  return INFAAS_OK;
}

}  // namespace

int infaas::record_cuda_error(cudaError_t e) { return cuda_fail(e); }

extern "C" {

int infaas_intpipe_probe(uint32_t iters, uint32_t *d_sink, int cuda_device, uint64_t *h_lane_ops,
                         void *cuda_stream) {
  if (!d_sink || !h_lane_ops) return INFAAS_E_NULL;
  if (iters == 0 || iters > (1u << 24)) return INFAAS_E_BAD_ARG;
  DeviceScope scope(cuda_device);
  if (scope.status != cudaSuccess) return cuda_fail(scope.status);
  const int sms = sm_count_of(cuda_device);
  if (sms <= 0) return cuda_fail(cudaErrorInvalidDevice);
  unsigned long long ops = 0;
  CUDA_TRY(infaas::launch_intpipe_probe(iters, 0x9E3779B1u, d_sink, sms, &ops, static_cast<cudaStream_t>(cuda_stream)));
  *h_lane_ops = ops;
  return INFAAS_OK;
}

const char *infaas_strerror(int code) {
  switch (code) {
    case INFAAS_OK: return "ok";
    case INFAAS_E_NULL: return "a required pointer is NULL";
    case INFAAS_E_BAD_TASK: return "row task out of range, or n_tasks is 0 or above 65535";
    case INFAAS_E_BAD_BATCH: return "row batch size is 0";
    case INFAAS_E_BAD_LAT: return "row latency is 0";
    case INFAAS_E_BAD_ACC: return "row accuracy above 10000 basis points, or reserved field not 0";
    case INFAAS_E_TOO_LARGE: return "size limit exceeded";
    case INFAAS_E_CUDA: return "CUDA call failed (see infaas_last_cuda_error)";
    case INFAAS_E_ALIGN: return "device array is not 16-byte aligned";
    case INFAAS_E_DEVICE: return "a kernel reported an internal error";
    case INFAAS_E_BAD_STATE: return "variant state is not one of INFAAS_STATE_*";
    case INFAAS_E_BAD_ARG: return "a scalar argument is out of range, or a required set-up call is missing";
    default: return "unknown error code";
  }
}

const char *infaas_last_cuda_error(void) { return g_cuda_error.c_str(); }

int infaas_catalog_load(const infaas_variant *rows, uint32_t n_variants, uint32_t n_tasks,
                        int cuda_device, infaas_catalog **out) {
  if (out) *out = nullptr;
  if (!rows || !out) return INFAAS_E_NULL;
  if (n_tasks == 0 || n_tasks > 65535u) return INFAAS_E_BAD_TASK;
  if (n_variants == 0 || n_variants > INFAAS_MAX_VARIANTS) return INFAAS_E_TOO_LARGE;

  // ---- validate and bucket by task (stable: ascending id inside a task) ----
  std::vector<uint32_t> task_off(n_tasks + 1, 0);
  uint32_t acc_min = 10000, acc_max = 0, lat_min = 0xFFFFFFFFu;
  for (uint32_t v = 0; v < n_variants; ++v) {
    const infaas_variant &r = rows[v];
    if (r.task >= n_tasks) return INFAAS_E_BAD_TASK;
    if (r.batch == 0) return INFAAS_E_BAD_BATCH;
    if (r.lat_us == 0) return INFAAS_E_BAD_LAT;
    if (r.acc_bp > 10000 || r.reserved != 0) return INFAAS_E_BAD_ACC;
    task_off[r.task + 1]++;
    if (r.acc_bp < acc_min) acc_min = r.acc_bp;
    if (r.acc_bp > acc_max) acc_max = r.acc_bp;
    if (r.lat_us < lat_min) lat_min = r.lat_us;
  }
  // the window of accuracies every bitmap of the index covers: whole words of 24 basis points
  const uint32_t acc_lo = acc_min / infaas::ACC_WORD_BITS * infaas::ACC_WORD_BITS;
  const uint32_t nbw = (acc_max + 1u - acc_lo) / infaas::ACC_WORD_BITS + 1u;
  uint32_t max_task = 0;
  for (uint32_t t = 0; t < n_tasks; ++t) {
    if (task_off[t + 1] > max_task) max_task = task_off[t + 1];
    task_off[t + 1] += task_off[t];
  }
  if (max_task > INFAAS_MAX_TASK_VARIANTS) return INFAAS_E_TOO_LARGE;
  std::vector<uint32_t> reg_off(n_tasks + 1, 0);
  uint64_t region_bytes = 0;
  for (uint32_t t = 0; t < n_tasks; ++t) {
    region_bytes += infaas::region_capacity(task_off[t + 1] - task_off[t]);
    if (region_bytes > 0xF0000000ull) return INFAAS_E_TOO_LARGE;
    reg_off[t + 1] = (uint32_t)region_bytes;
  }

  std::vector<uint32_t> h_lat(n_variants), h_cost(n_variants), h_id(n_variants), h_queued(n_variants),
      slot_of_id(n_variants);
  std::vector<uint16_t> h_batch(n_variants), h_acc(n_variants), h_arch(n_variants);
  std::vector<unsigned long long> h_qps(n_variants);
  {
    std::vector<uint32_t> cursor(task_off.begin(), task_off.end() - 1);
    for (uint32_t v = 0; v < n_variants; ++v) {
      const infaas_variant &r = rows[v];
      const uint32_t s = cursor[r.task]++;
      h_lat[s] = r.lat_us; h_batch[s] = r.batch; h_acc[s] = r.acc_bp; h_cost[s] = r.cost;
      h_id[s] = v; h_queued[s] = r.queued; slot_of_id[v] = s; h_arch[s] = r.arch;
      h_qps[s] = 1000000000ull * r.batch / r.lat_us;     // floor(10^9 * batch / lat_us)
    }
  }

  infaas_catalog *c = new (std::nothrow) infaas_catalog();
  if (!c) return INFAAS_E_TOO_LARGE;
  c->device = cuda_device;
  DeviceScope scope(cuda_device);
  if (scope.status != cudaSuccess) { delete c; return cuda_fail(scope.status); }

  // ---- one arena, carved into 256-byte aligned arrays ----
  // lists longer than the index supports are cut into segments; every segment but a task's
  // first needs a header and parameters outside the image
  uint64_t worst_image = infaas::image_var_offset(n_tasks, nbw);
  std::vector<uint32_t> seg_base(n_tasks + 1, 0);
  for (uint32_t t = 0; t < n_tasks; ++t) {
    const uint32_t V = task_off[t + 1] - task_off[t];
    // a state-aware catalog has two lists per task (V entries together): one segment more
    const uint32_t segs = (V + infaas::INDEX_MAX_F - 1) / infaas::INDEX_MAX_F + 1;
    seg_base[t + 1] = seg_base[t] + segs - 1;
    worst_image += (uint64_t)segs * infaas::block_capacity(V, nbw);
  }
  const uint32_t n_extra = seg_base[n_tasks];
  if (worst_image > 0xFFFFFFF0ull) { delete c; return INFAAS_E_TOO_LARGE; }
  size_t total = 0;
  auto carve = [&total](size_t bytes) { size_t off = total; total += round_up(bytes, 256); return off; };
  const size_t o_task_off = carve((n_tasks + 1) * 4), o_reg_off = carve((n_tasks + 1) * 4);
  const size_t o_lat = carve((size_t)n_variants * 4), o_batch = carve((size_t)n_variants * 2);
  const size_t o_acc = carve((size_t)n_variants * 2), o_cost = carve((size_t)n_variants * 4);
  const size_t o_id = carve((size_t)n_variants * 4), o_queued = carve((size_t)n_variants * 4);
  const size_t o_pred = carve((size_t)n_variants * 4), o_served = carve((size_t)n_variants * 8);
  const size_t o_count = carve((size_t)n_variants * 4);
  const size_t o_state = carve((size_t)n_variants), o_load_lat = carve((size_t)n_variants * 4);
  const size_t o_inst = carve((size_t)n_variants * 4), o_arch = carve((size_t)n_variants * 2);
  const size_t o_task_slo = carve((size_t)n_tasks * 4), o_qps = carve((size_t)n_variants * 8);
  const size_t o_hw = carve((size_t)n_variants), o_worker_of = carve((size_t)n_variants * 4);
  const size_t o_best_inst = carve((size_t)n_variants * 8), o_best_hw = carve(256 * 8);
  const size_t o_regions = carve((size_t)region_bytes);
  const size_t o_flen = carve((size_t)n_tasks * 4), o_slow = carve(((size_t)n_tasks + n_extra) * 16);
  const size_t o_seg_base = carve((n_tasks + 1) * 4), o_xhdr = carve((size_t)n_extra * 16 + 16);
  const size_t o_image = carve((size_t)worst_image), o_hdr = carve(16);
  const size_t o_counters = carve(24), o_rebuild = carve(32), o_err = carve(4), o_seen = carve(4);

#define LOAD_TRY(expr)                                                     \
  do {                                                                     \
    cudaError_t e__ = (expr);                                              \
    if (e__ != cudaSuccess) { infaas_catalog_free(c); return cuda_fail(e__); } \
  } while (0)

  cudaDeviceProp prop;
  LOAD_TRY(cudaGetDeviceProperties(&prop, cuda_device));
  c->sm_count = prop.multiProcessorCount;
  LOAD_TRY(cudaMalloc(&c->arena, total));
  unsigned char *base = static_cast<unsigned char *>(c->arena);
  LOAD_TRY(cudaMemset(base, 0, total));
  LOAD_TRY(cudaMemset(base + o_state, INFAAS_STATE_ACTIVE, n_variants));
  LOAD_TRY(cudaMemcpy(base + o_task_off, task_off.data(), (n_tasks + 1) * 4, cudaMemcpyHostToDevice));
  LOAD_TRY(cudaMemcpy(base + o_reg_off, reg_off.data(), (n_tasks + 1) * 4, cudaMemcpyHostToDevice));
  LOAD_TRY(cudaMemcpy(base + o_seg_base, seg_base.data(), (n_tasks + 1) * 4, cudaMemcpyHostToDevice));
  LOAD_TRY(cudaMemcpy(base + o_lat, h_lat.data(), (size_t)n_variants * 4, cudaMemcpyHostToDevice));
  LOAD_TRY(cudaMemcpy(base + o_batch, h_batch.data(), (size_t)n_variants * 2, cudaMemcpyHostToDevice));
  LOAD_TRY(cudaMemcpy(base + o_acc, h_acc.data(), (size_t)n_variants * 2, cudaMemcpyHostToDevice));
  LOAD_TRY(cudaMemcpy(base + o_cost, h_cost.data(), (size_t)n_variants * 4, cudaMemcpyHostToDevice));
  LOAD_TRY(cudaMemcpy(base + o_id, h_id.data(), (size_t)n_variants * 4, cudaMemcpyHostToDevice));
  LOAD_TRY(cudaMemcpy(base + o_queued, h_queued.data(), (size_t)n_variants * 4, cudaMemcpyHostToDevice));
  LOAD_TRY(cudaMemcpy(base + o_arch, h_arch.data(), (size_t)n_variants * 2, cudaMemcpyHostToDevice));
  LOAD_TRY(cudaMemcpy(base + o_qps, h_qps.data(), (size_t)n_variants * 8, cudaMemcpyHostToDevice));
  c->s_qps = reinterpret_cast<unsigned long long *>(base + o_qps);
  {
    std::vector<unsigned char> h_hw(n_variants);
    for (uint32_t v = 0; v < n_variants; ++v) h_hw[v] = rows[v].hw;
    LOAD_TRY(cudaMemcpy(base + o_hw, h_hw.data(), n_variants, cudaMemcpyHostToDevice));
  }
  c->hw_by_id = base + o_hw;
  c->worker_of = reinterpret_cast<uint32_t *>(base + o_worker_of);
  c->best_inst = reinterpret_cast<unsigned long long *>(base + o_best_inst);
  c->best_hw = reinterpret_cast<unsigned long long *>(base + o_best_hw);
  c->s_inst = reinterpret_cast<uint32_t *>(base + o_inst);
  c->s_arch = reinterpret_cast<uint16_t *>(base + o_arch);
  c->task_slo = reinterpret_cast<uint32_t *>(base + o_task_slo);

  DeviceCatalog &d = c->d;
  d.n_variants = n_variants;
  d.n_tasks = n_tasks;
  d.max_task_variants = max_task;
  d.task_off = reinterpret_cast<const uint32_t *>(base + o_task_off);
  d.reg_off = reinterpret_cast<const uint32_t *>(base + o_reg_off);
  d.s_lat = reinterpret_cast<const uint32_t *>(base + o_lat);
  d.s_batch = reinterpret_cast<const uint16_t *>(base + o_batch);
  d.s_acc = reinterpret_cast<const uint16_t *>(base + o_acc);
  d.s_cost = reinterpret_cast<const uint32_t *>(base + o_cost);
  d.s_id = reinterpret_cast<const uint32_t *>(base + o_id);
  d.s_queued = reinterpret_cast<uint32_t *>(base + o_queued);
  d.s_pred = reinterpret_cast<uint32_t *>(base + o_pred);
  d.s_served = reinterpret_cast<unsigned long long *>(base + o_served);
  d.count_by_id = reinterpret_cast<uint32_t *>(base + o_count);
  d.stateful = 0;
  d.s_state = base + o_state;
  d.s_load_lat = reinterpret_cast<const uint32_t *>(base + o_load_lat);
  d.regions = base + o_regions;
  d.f_len = reinterpret_cast<uint32_t *>(base + o_flen);
  d.slow = reinterpret_cast<uint4 *>(base + o_slow);
  d.seg_base = reinterpret_cast<const uint32_t *>(base + o_seg_base);
  d.xhdr = reinterpret_cast<uint4 *>(base + o_xhdr);
  d.image = base + o_image;
  d.image_capacity = (uint32_t)worst_image;
  d.image_hdr = reinterpret_cast<uint32_t *>(base + o_hdr);
  d.acc_lo = acc_lo;
  d.nbw = nbw;
  d.lat_code_lo = float_bits_rz(lat_min) >> 16;
  d.counters = reinterpret_cast<unsigned long long *>(base + o_counters);
  d.alloc_ctr = reinterpret_cast<unsigned long long *>(base + o_rebuild);
  d.err = reinterpret_cast<uint32_t *>(base + o_err);
  d.slo_seen = reinterpret_cast<uint32_t *>(base + o_seen);
  c->slot_of_id.swap(slot_of_id);
  c->task_off.swap(task_off);
  c->reg_off.swap(reg_off);
  c->worst_image_bytes = (uint32_t)worst_image;

  LOAD_TRY(infaas::prepare_select_kernel());
  LOAD_TRY(infaas::prepare_rebuild_kernel());
  LOAD_TRY(infaas::launch_rebuild(d, /*advance_queues=*/false, 0, nullptr));
  LOAD_TRY(cudaDeviceSynchronize());
  int rc = refresh_select_plan(c, nullptr);
  if (rc != INFAAS_OK) { infaas_catalog_free(c); return rc; }
#undef LOAD_TRY
  *out = c;
  return INFAAS_OK;
}

int infaas_select_batch(infaas_catalog *c, const uint16_t *d_task, const uint32_t *d_slo_us,
                        const uint16_t *d_min_acc_bp, uint64_t n, uint32_t *d_decision,
                        void *cuda_stream) {
  if (!c) return INFAAS_E_NULL;
  if (n == 0) return INFAAS_OK;
  if (!d_task || !d_slo_us || !d_min_acc_bp || !d_decision) return INFAAS_E_NULL;
  if (!aligned16(d_task) || !aligned16(d_slo_us) || !aligned16(d_min_acc_bp) || !aligned16(d_decision))
    return INFAAS_E_ALIGN;
  DeviceScope scope(c->device);
  if (scope.status != cudaSuccess) return cuda_fail(scope.status);
  CUDA_TRY(infaas::launch_select(c->d, d_task, d_slo_us, d_min_acc_bp, n, d_decision, c->sm_count,
                                 c->select_smem, /*tally=*/false, static_cast<cudaStream_t>(cuda_stream)));
  return INFAAS_OK;
}

int infaas_select_update(infaas_catalog *c, const uint16_t *d_task, const uint32_t *d_slo_us,
                         const uint16_t *d_min_acc_bp, uint64_t n, uint32_t *d_decision,
                         uint32_t window_us, void *cuda_stream) {
  if (!c) return INFAAS_E_NULL;
  if (n > 0xFFFFFFFFull) return INFAAS_E_TOO_LARGE;
  if (n == 0 || n >= infaas::FUSED_TALLY_MAX_N) {
    // large batches: a pass of its own over the decisions with shared-memory histograms is cheaper
    const int rc = infaas_select_batch(c, d_task, d_slo_us, d_min_acc_bp, n, d_decision, cuda_stream);
    return rc != INFAAS_OK ? rc : infaas_load_update(c, d_decision, n, window_us, cuda_stream);
  }
  if (!d_task || !d_slo_us || !d_min_acc_bp || !d_decision) return INFAAS_E_NULL;
  if (!aligned16(d_task) || !aligned16(d_slo_us) || !aligned16(d_min_acc_bp) || !aligned16(d_decision))
    return INFAAS_E_ALIGN;
  DeviceScope scope(c->device);
  if (scope.status != cudaSuccess) return cuda_fail(scope.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  CUDA_TRY(infaas::launch_select(c->d, d_task, d_slo_us, d_min_acc_bp, n, d_decision, c->sm_count,
                                 c->select_smem, /*tally=*/true, s));
  CUDA_TRY(infaas::launch_rebuild(c->d, /*advance_queues=*/true, window_us, s));
  return INFAAS_OK;
}

int infaas_tally(infaas_catalog *c, const uint32_t *d_decision, uint64_t n, void *cuda_stream) {
  if (!c) return INFAAS_E_NULL;
  if (n > 0xFFFFFFFFull) return INFAAS_E_TOO_LARGE;
  if (n > 0 && !d_decision) return INFAAS_E_NULL;
  if (n > 0 && !aligned16(d_decision)) return INFAAS_E_ALIGN;
  DeviceScope scope(c->device);
  if (scope.status != cudaSuccess) return cuda_fail(scope.status);
  CUDA_TRY(infaas::launch_tally(c->d, d_decision, n, c->sm_count, static_cast<cudaStream_t>(cuda_stream)));
  return INFAAS_OK;
}

int infaas_pending_counts(infaas_catalog *c, uint32_t *d_counts, int set, void *cuda_stream) {
  if (!c || !d_counts) return INFAAS_E_NULL;
  if (!aligned16(d_counts)) return INFAAS_E_ALIGN;
  DeviceScope scope(c->device);
  if (scope.status != cudaSuccess) return cuda_fail(scope.status);
  const size_t bytes = (size_t)c->d.n_variants * 4;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (set) CUDA_TRY(cudaMemcpyAsync(c->d.count_by_id, d_counts, bytes, cudaMemcpyDeviceToDevice, s));
  else CUDA_TRY(cudaMemcpyAsync(d_counts, c->d.count_by_id, bytes, cudaMemcpyDeviceToDevice, s));
  return INFAAS_OK;
}

int infaas_advance(infaas_catalog *c, uint32_t window_us, void *cuda_stream) {
  if (!c) return INFAAS_E_NULL;
  DeviceScope scope(c->device);
  if (scope.status != cudaSuccess) return cuda_fail(scope.status);
  CUDA_TRY(infaas::launch_rebuild(c->d, /*advance_queues=*/true, window_us, static_cast<cudaStream_t>(cuda_stream)));
  return INFAAS_OK;
}

int infaas_load_update(infaas_catalog *c, const uint32_t *d_decision, uint64_t n,
                       uint32_t window_us, void *cuda_stream) {
  const int rc = infaas_tally(c, d_decision, n, cuda_stream);
  return rc != INFAAS_OK ? rc : infaas_advance(c, window_us, cuda_stream);
}

int infaas_catalog_set_states(infaas_catalog *c, const uint8_t *h_state, const uint32_t *h_load_lat_us,
                              void *cuda_stream) {
  if (!c || !h_state) return INFAAS_E_NULL;
  const uint32_t nv = c->d.n_variants;
  for (uint32_t v = 0; v < nv; ++v)
    if (h_state[v] > INFAAS_STATE_INTERFERED) return INFAAS_E_BAD_STATE;
  DeviceScope scope(c->device);
  if (scope.status != cudaSuccess) return cuda_fail(scope.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  std::vector<unsigned char> st(nv);
  std::vector<uint32_t> ll(nv, 0u);
  for (uint32_t v = 0; v < nv; ++v) {
    st[c->slot_of_id[v]] = h_state[v];
    if (h_load_lat_us) ll[c->slot_of_id[v]] = h_load_lat_us[v];
  }
  CUDA_TRY(cudaMemcpyAsync(c->d.s_state, st.data(), nv, cudaMemcpyHostToDevice, s));
  CUDA_TRY(cudaMemcpyAsync(const_cast<uint32_t *>(c->d.s_load_lat), ll.data(), (size_t)nv * 4,
                           cudaMemcpyHostToDevice, s));
  c->d.stateful = 1;
  CUDA_TRY(infaas::launch_rebuild(c->d, /*advance_queues=*/false, 0, s));
  CUDA_TRY(cudaStreamSynchronize(s));     // the host copies above go out of scope
  return refresh_select_plan(c, s);
}

int infaas_catalog_get_states(infaas_catalog *c, uint8_t *h_state, void *cuda_stream) {
  if (!c || !h_state) return INFAAS_E_NULL;
  DeviceScope scope(c->device);
  if (scope.status != cudaSuccess) return cuda_fail(scope.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const uint32_t nv = c->d.n_variants;
  std::vector<unsigned char> st(nv);
  CUDA_TRY(cudaMemcpyAsync(st.data(), c->d.s_state, nv, cudaMemcpyDeviceToHost, s));
  CUDA_TRY(cudaStreamSynchronize(s));
  for (uint32_t v = 0; v < nv; ++v) h_state[v] = st[c->slot_of_id[v]];
  return INFAAS_OK;
}

int infaas_autoscale_config(infaas_catalog *c, const uint32_t *h_instances, const uint32_t *h_task_slo_us,
                            void *cuda_stream) {
  if (!c || !h_instances || !h_task_slo_us) return INFAAS_E_NULL;
  DeviceScope scope(c->device);
  if (scope.status != cudaSuccess) return cuda_fail(scope.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const uint32_t nv = c->d.n_variants;
  std::vector<uint32_t> inst(nv);
  for (uint32_t v = 0; v < nv; ++v) inst[c->slot_of_id[v]] = h_instances[v];
  CUDA_TRY(cudaMemcpyAsync(c->s_inst, inst.data(), (size_t)nv * 4, cudaMemcpyHostToDevice, s));
  CUDA_TRY(cudaMemcpyAsync(c->task_slo, h_task_slo_us, (size_t)c->d.n_tasks * 4, cudaMemcpyHostToDevice, s));
  CUDA_TRY(cudaStreamSynchronize(s));
  c->autoscale_ready = true;
  return INFAAS_OK;
}

int infaas_autoscale_step(infaas_catalog *c, uint32_t window_us, uint32_t slack_pct, uint32_t lambda_milli,
                          uint32_t *d_variant, uint32_t *d_delta, void *cuda_stream) {
  if (!c || !d_variant || !d_delta) return INFAAS_E_NULL;
  if (window_us == 0 || !c->autoscale_ready) return INFAAS_E_BAD_ARG;
  DeviceScope scope(c->device);
  if (scope.status != cudaSuccess) return cuda_fail(scope.status);
  CUDA_TRY(infaas::launch_autoscale(c->d, c->s_inst, c->s_arch, c->s_qps, c->task_slo, window_us, slack_pct, lambda_milli,
                                    d_variant, d_delta, static_cast<cudaStream_t>(cuda_stream)));
  return INFAAS_OK;
}

int infaas_workers_config(infaas_catalog *c, const uint32_t *h_inst_variant, const uint32_t *h_inst_worker,
                          const uint32_t *h_inst_load, uint32_t n_inst, const uint8_t *h_worker_hw,
                          const uint32_t *h_worker_util, uint32_t n_workers, void *cuda_stream) {
  if (!c) return INFAAS_E_NULL;
  if (n_inst && (!h_inst_variant || !h_inst_worker || !h_inst_load)) return INFAAS_E_NULL;
  if (n_workers && (!h_worker_hw || !h_worker_util)) return INFAAS_E_NULL;
  DeviceScope scope(c->device);
  if (scope.status != cudaSuccess) return cuda_fail(scope.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  // one temporary buffer: three u32 arrays of n_inst, one u32 array and one u8 array of n_workers
  const size_t ib = round_up((size_t)n_inst * 4, 256), wb = round_up((size_t)n_workers * 4, 256);
  unsigned char *tmp = nullptr;
  CUDA_TRY(cudaMalloc(&tmp, 3 * ib + 2 * wb + 256));
  uint32_t *d_iv = reinterpret_cast<uint32_t *>(tmp), *d_iw = reinterpret_cast<uint32_t *>(tmp + ib),
           *d_il = reinterpret_cast<uint32_t *>(tmp + 2 * ib), *d_wu = reinterpret_cast<uint32_t *>(tmp + 3 * ib);
  unsigned char *d_wh = tmp + 3 * ib + wb;
  cudaError_t e = cudaSuccess;
  auto up = [&](void *dst, const void *src, size_t bytes) {
    if (e == cudaSuccess && bytes) e = cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, s);
  };
  up(d_iv, h_inst_variant, (size_t)n_inst * 4);
  up(d_iw, h_inst_worker, (size_t)n_inst * 4);
  up(d_il, h_inst_load, (size_t)n_inst * 4);
  up(d_wu, h_worker_util, (size_t)n_workers * 4);
  up(d_wh, h_worker_hw, (size_t)n_workers);
  if (e == cudaSuccess)
    e = infaas::launch_workers_build(c->d.n_variants, c->hw_by_id, d_iv, d_iw, d_il, n_inst, d_wh, d_wu, n_workers,
                                     c->best_inst, c->best_hw, c->worker_of, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  (void)cudaFree(tmp);
  if (e != cudaSuccess) return cuda_fail(e);
  c->workers_ready = true;
  return INFAAS_OK;
}

int infaas_assign_workers(infaas_catalog *c, const uint32_t *d_decision, uint64_t n, uint32_t *d_worker,
                          void *cuda_stream) {
  if (!c) return INFAAS_E_NULL;
  if (!c->workers_ready) return INFAAS_E_BAD_ARG;
  if (n == 0) return INFAAS_OK;
  if (!d_decision || !d_worker) return INFAAS_E_NULL;
  if (!aligned16(d_decision) || !aligned16(d_worker)) return INFAAS_E_ALIGN;
  DeviceScope scope(c->device);
  if (scope.status != cudaSuccess) return cuda_fail(scope.status);
  CUDA_TRY(infaas::launch_assign_workers(d_decision, n, c->d.n_variants, c->worker_of, d_worker, c->sm_count,
                                         static_cast<cudaStream_t>(cuda_stream)));
  return INFAAS_OK;
}

int infaas_catalog_get_state(infaas_catalog *c, uint32_t *h_queued, uint32_t *h_pred_lat_us,
                             uint64_t *h_served_total, uint64_t h_counters[3], void *cuda_stream) {
  if (!c) return INFAAS_E_NULL;
  DeviceScope scope(c->device);
  if (scope.status != cudaSuccess) return cuda_fail(scope.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const uint32_t nv = c->d.n_variants;
  std::vector<uint32_t> tmp32;
  std::vector<unsigned long long> tmp64;
  if (h_queued) {
    tmp32.resize(nv);
    CUDA_TRY(cudaMemcpyAsync(tmp32.data(), c->d.s_queued, (size_t)nv * 4, cudaMemcpyDeviceToHost, s));
    CUDA_TRY(cudaStreamSynchronize(s));
    for (uint32_t v = 0; v < nv; ++v) h_queued[v] = tmp32[c->slot_of_id[v]];
  }
  if (h_pred_lat_us) {
    tmp32.resize(nv);
    CUDA_TRY(cudaMemcpyAsync(tmp32.data(), c->d.s_pred, (size_t)nv * 4, cudaMemcpyDeviceToHost, s));
    CUDA_TRY(cudaStreamSynchronize(s));
    for (uint32_t v = 0; v < nv; ++v) h_pred_lat_us[v] = tmp32[c->slot_of_id[v]];
  }
  if (h_served_total) {
    tmp64.resize(nv);
    CUDA_TRY(cudaMemcpyAsync(tmp64.data(), c->d.s_served, (size_t)nv * 8, cudaMemcpyDeviceToHost, s));
    CUDA_TRY(cudaStreamSynchronize(s));
    for (uint32_t v = 0; v < nv; ++v) h_served_total[v] = tmp64[c->slot_of_id[v]];
  }
  if (h_counters) {
    unsigned long long k[3];
    CUDA_TRY(cudaMemcpyAsync(k, c->d.counters, sizeof(k), cudaMemcpyDeviceToHost, s));
    CUDA_TRY(cudaStreamSynchronize(s));
    for (int i = 0; i < 3; ++i) h_counters[i] = k[i];
  }
  uint32_t err = 0;
  CUDA_TRY(cudaMemcpyAsync(&err, c->d.err, 4, cudaMemcpyDeviceToHost, s));
  CUDA_TRY(cudaStreamSynchronize(s));
  int rc = refresh_select_plan(c, s);
  if (rc != INFAAS_OK) return rc;
  if (err != infaas::DEV_ERR_NONE) {
    CUDA_TRY(cudaMemsetAsync(c->d.err, 0, 4, s));
    CUDA_TRY(cudaStreamSynchronize(s));
    return INFAAS_E_DEVICE;
  }
  return INFAAS_OK;
}

int infaas_catalog_get_frontier(infaas_catalog *c, uint32_t task, uint32_t *h_ids, uint32_t cap,
                                uint32_t *h_len, void *cuda_stream) {
  if (!c || !h_len) return INFAAS_E_NULL;
  if (task >= c->d.n_tasks) return INFAAS_E_BAD_TASK;
  DeviceScope scope(c->device);
  if (scope.status != cudaSuccess) return cuda_fail(scope.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  uint32_t len = 0;
  CUDA_TRY(cudaMemcpyAsync(&len, c->d.f_len + task, 4, cudaMemcpyDeviceToHost, s));
  CUDA_TRY(cudaStreamSynchronize(s));
  *h_len = len;
  const uint32_t ncopy = len < cap ? len : cap;
  if (h_ids && ncopy) {
    const uint32_t V = c->task_off[task + 1] - c->task_off[task];
    const unsigned char *ids = c->d.regions + c->reg_off[task] + 8u * (size_t)V;
    CUDA_TRY(cudaMemcpyAsync(h_ids, ids, (size_t)ncopy * 4, cudaMemcpyDeviceToHost, s));
    CUDA_TRY(cudaStreamSynchronize(s));
  }
  return INFAAS_OK;
}

int infaas_catalog_get_info(infaas_catalog *c, uint32_t h_info[8], void *cuda_stream) {
  if (!c || !h_info) return INFAAS_E_NULL;
  DeviceScope scope(c->device);
  if (scope.status != cudaSuccess) return cuda_fail(scope.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  // the image size comes from the rebuild kernel; the list statistics are summed up here
  // from the per-task lengths and flags (reporting only)
  const uint32_t T = c->d.n_tasks;
  uint32_t bytes = 0;
  std::vector<uint32_t> f_len(T);
  std::vector<uint4> slow(T);
  CUDA_TRY(cudaMemcpyAsync(&bytes, c->d.image_hdr, 4, cudaMemcpyDeviceToHost, s));
  CUDA_TRY(cudaMemcpyAsync(f_len.data(), c->d.f_len, (size_t)T * 4, cudaMemcpyDeviceToHost, s));
  CUDA_TRY(cudaMemcpyAsync(slow.data(), c->d.slow, (size_t)T * 16, cudaMemcpyDeviceToHost, s));
  CUDA_TRY(cudaStreamSynchronize(s));
  h_info[0] = bytes;
  h_info[1] = h_info[2] = h_info[3] = 0;
  for (uint32_t t = 0; t < T; ++t) {
    if (f_len[t] > h_info[1]) h_info[1] = f_len[t];
    h_info[2] += f_len[t];
    if (f_len[t] > 0 && (slow[t].z & infaas::TASK_FLAG_NOT_INDEXED)) ++h_info[3];
  }
  h_info[4] = infaas::select_image_smem(c->select_smem);
  h_info[5] = h_info[6] = h_info[7] = 0;
  return INFAAS_OK;
}

void infaas_catalog_free(infaas_catalog *c) {
  if (!c) return;
  if (c->arena) {
    DeviceScope scope(c->device);
    (void)cudaFree(c->arena);
  }
  delete c;
}

}  // extern "C"
