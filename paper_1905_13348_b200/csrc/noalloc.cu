// Tally entry point that allocates nothing: its scratch is a fixed array in the library's
// device image instead of memory obtained at run time.
#include <mutex>

#include "common.cuh"

namespace {

// counts for up to INFAAS_STATIC_MAX_VARIANTS variants, then three 64-bit counters
struct StaticScratch {
  uint32_t count[INFAAS_STATIC_MAX_VARIANTS];
  unsigned long long counters[4];
};
static __device__ __align__(256) StaticScratch g_tally_scratch;

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
StaticScratch *g_scratch_addr[kMaxDevices] = {};   // device address of the array, per device
int g_sm_count[kMaxDevices] = {};                  // multiprocessors, per device

}  // namespace

extern "C" int infaas_tally_static(const uint32_t *d_decision, uint64_t n, uint32_t n_variants,
                                   uint32_t *d_count, uint64_t *d_counters, int cuda_device,
                                   void *cuda_stream) {
  if (!d_count || !d_counters || (n > 0 && !d_decision)) return INFAAS_E_NULL;
  if (n_variants == 0 || n_variants > INFAAS_STATIC_MAX_VARIANTS || n > 0xFFFFFFFFull)
    return INFAAS_E_TOO_LARGE;
  if (n > 0 && (reinterpret_cast<uintptr_t>(d_decision) & 15u)) return INFAAS_E_ALIGN;
  if (cuda_device < 0 || cuda_device >= kMaxDevices) return INFAAS_E_TOO_LARGE;

  int prev = -1;
  cudaError_t e = cudaGetDevice(&prev);
  if (e != cudaSuccess) return infaas::record_cuda_error(e);
  if (prev != cuda_device && (e = cudaSetDevice(cuda_device)) != cudaSuccess) return infaas::record_cuda_error(e);
  int rc = INFAAS_OK;
  StaticScratch *scratch = nullptr;
  {
    // The array's name is only a host-side stand-in; the kernels need its address on this
    // device, looked up once per device while that device is current.
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[cuda_device]) {
      void *p = nullptr;
      int sms = 0;
      // (the tally kernels' shared-memory limit is a per-device attribute, set here too)
      if ((e = cudaGetSymbolAddress(&p, g_tally_scratch)) != cudaSuccess ||
          (e = infaas::prepare_rebuild_kernel()) != cudaSuccess ||
          (e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, cuda_device)) != cudaSuccess) {
        rc = infaas::record_cuda_error(e);
      } else if (!p || sms <= 0) {
        rc = infaas::record_cuda_error(cudaErrorInvalidSymbol);
      } else {
        g_scratch_addr[cuda_device] = static_cast<StaticScratch *>(p);
        g_sm_count[cuda_device] = sms;
      }
    }
    scratch = g_scratch_addr[cuda_device];
  }
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (rc == INFAAS_OK) {
    // every call shares the array and finds the previous call's numbers in it: clear first
    infaas::DeviceCatalog view{};
    view.n_variants = n_variants;
    view.count_by_id = scratch->count;
    view.counters = scratch->counters;
    if ((e = cudaMemsetAsync(scratch, 0, (size_t)n_variants * 4, s)) != cudaSuccess ||
        (e = cudaMemsetAsync(scratch->counters, 0, sizeof(scratch->counters), s)) != cudaSuccess ||
        (e = infaas::launch_tally(view, d_decision, n, g_sm_count[cuda_device], s)) != cudaSuccess ||
        (e = cudaMemcpyAsync(d_count, scratch->count, (size_t)n_variants * 4, cudaMemcpyDeviceToDevice, s)) != cudaSuccess ||
        (e = cudaMemcpyAsync(d_counters, scratch->counters, 24, cudaMemcpyDeviceToDevice, s)) != cudaSuccess)
      rc = infaas::record_cuda_error(e);   // the text is kept for infaas_last_cuda_error()
  }
  if (prev != cuda_device) (void)cudaSetDevice(prev);
  return rc;
}
