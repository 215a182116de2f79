// lite3r_sla_forward_static_scratch: the SLA forward for callers that cannot hand the library any scratch buffer.
//
// Some hosts of this library cannot allocate device memory at the point where they call it: a plug-in running inside
// another runtime's pre-planned arena, a real-time loop that must not touch the allocator, or a process whose memory
// pool has already been sized to the last byte.  For them the
// forward's scratch (per-key-block summaries and per-query-block aggregates) lives in a fixed array that is part of
// the loaded library image.  CUDA loads a module's device code lazily by default, so the array takes its
// LITE3R_STATIC_SCRATCH_BYTES of device memory when this file's module is first touched on a device -- the first
// call of the entry point there -- and keeps them until the process exits; every later call allocates nothing.
// The paper has no counterpart; this is a deployment convenience of the library.
#include <mutex>

#include "common.cuh"

namespace lite3r {
namespace {

static __device__ __align__(256) unsigned char g_static_scratch[LITE3R_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_ptr[kMaxDevices] = {};

// In host code `g_static_scratch` is only a handle for the symbol, not a device address, so the address each device
// gave the array is looked up once per device (with that device current) and cached.
lite3r_status scratch_address(void** ptr) {
  int device = -1;
  lite3r_status st = record_cuda(cudaGetDevice(&device));
  if (st != LITE3R_OK) return st;
  if (device < 0 || device >= kMaxDevices) return LITE3R_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_scratch_ptr[device] == nullptr) {
    void* p = nullptr;
    st = record_cuda(cudaGetSymbolAddress(&p, g_static_scratch));
    if (st != LITE3R_OK) return st;
    if (p == nullptr) return LITE3R_ERR_CUDA;
    g_scratch_ptr[device] = p;
  }
  *ptr = g_scratch_ptr[device];
  return LITE3R_OK;
}

}  // namespace
}  // namespace lite3r

extern "C" lite3r_status lite3r_sla_forward_static_scratch(const lite3r_fp8* q, const lite3r_fp8* k,
                                                           const lite3r_fp8* v, const float* proj,
                                                           long long proj_head_stride, const lite3r_shape* shape,
                                                           lite3r_phi phi, const lite3r_plan* plan, void* out,
                                                           lite3r_dtype out_dtype, long long out_stride_b,
                                                           long long out_stride_h, long long out_stride_n,
                                                           int* device_status, void* stream) {
  using namespace lite3r;
  if (shape == nullptr || plan == nullptr) return LITE3R_ERR_INVALID_ARG;
  // The array's address is resolved first, before any other check: under lazy module loading this look-up is what
  // loads the module that holds the array (and makes the driver set its 32 MiB aside), so even a call that is then
  // refused for its size serves as the warm-up that start-up code should make once per device.
  void* scratch = nullptr;
  lite3r_status st = scratch_address(&scratch);
  if (st != LITE3R_OK) return st;
  size_t need = 0;
  st = lite3r_forward_workspace(shape, 0.0, 0.0, &need);  // validates the shape
  if (st != LITE3R_OK) return st;
  need = forward_workspace_bytes(*shape, Counts{plan->k_crit, plan->k_marg, plan->k_neg});
  if (need > static_cast<size_t>(LITE3R_STATIC_SCRATCH_BYTES)) return LITE3R_ERR_WORKSPACE;
  return lite3r_sla_forward(q, k, v, proj, proj_head_stride, shape, 0.0, 0.0, phi, plan, out, out_dtype, out_stride_b,
                            out_stride_h, out_stride_n, scratch, static_cast<size_t>(LITE3R_STATIC_SCRATCH_BYTES),
                            device_status, stream);
}
