// cmoe_route_static: two-stage routing without a handle, an arena or any allocation.
//
// cmoe_route reads the router matrices from the arena the caller allocated for cmoe_create, where
// they sit re-laid-out one row per cluster / expert.  Some callers cannot provide such an arena: a
// plugin running inside a host application whose memory pool is frozen after start-up, or a
// dispatcher thread that must decide where a token goes before any layer handle exists.  For them
// this file keeps the re-laid-out router in a fixed device array that is part of the library image,
// and runs the same router kernel on it.
//
// The array is shared by every call on a device and keeps the previous call's contents, so each
// call rewrites every part it later reads (matrices, biases - zeros when none are given - and the
// label table).  Two calls whose GPU work overlaps (different streams) race on it.
#include <mutex>

#include "cmoe_internal.h"

namespace {

constexpr size_t kStaticBytes = CMOE_ROUTE_STATIC_BYTES;

// File-scope device storage: every GPU that loads the library holds these bytes until exit.
static __device__ __align__(256) unsigned char g_route_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
unsigned char* g_scratch_addr[kMaxDevices];   // device address of g_route_scratch, per device
bool g_scratch_ready[kMaxDevices];

// In host code `g_route_scratch` is only a stand-in for the symbol, not a device address; the real
// address differs per device and has to be asked for with that device current.
cudaError_t scratch_address(unsigned char** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_scratch_ready[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_route_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_addr[dev] = static_cast<unsigned char*>(p);
    g_scratch_ready[dev] = true;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

__global__ void iota_kernel(int* __restrict__ v, int n) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) v[i] = i;
}

size_t align256(size_t v) { return (v + 255) / 256 * 256; }

}  // namespace

extern "C" int cmoe_route_static(int32_t d, int32_t E, int32_t G, int32_t k,
                                 const float* C, const float* R, const float* b_c, const float* b_e,
                                 const void* x, int32_t T,
                                 int32_t* cluster_id, int32_t* expert_ids, float* gates,
                                 void* cuda_stream) {
  using namespace cmoe;
  if (d <= 0 || E <= 0 || G <= 0 || k <= 0 || T < 0) return CMOE_ERR_INVALID_ARG;
  if (E % G) return CMOE_ERR_UNSUPPORTED_SHAPE;
  const int K = E / G;
  if (G > kMaxG || K > kMaxK || k > K || k > kMaxKsel || d % 32) return CMOE_ERR_UNSUPPORTED_SHAPE;
  // layout inside the fixed array: Ct [G][d] | Rt [E][d] | bc [G] | be [E] | label [E]
  const size_t off_ct = 0;
  const size_t off_rt = align256(off_ct + sizeof(float) * (size_t)G * d);
  const size_t off_bc = align256(off_rt + sizeof(float) * (size_t)E * d);
  const size_t off_be = align256(off_bc + sizeof(float) * (size_t)G);
  const size_t off_lb = align256(off_be + sizeof(float) * (size_t)E);
  const size_t need = align256(off_lb + sizeof(int) * (size_t)E);
  if (need > kStaticBytes) return CMOE_ERR_WORKSPACE_TOO_SMALL;   // router larger than the fixed array
  if (T == 0) return CMOE_OK;
  if (!C || !R || !x || !cluster_id || !expert_ids || !gates) return CMOE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(x) & 15) != 0) return CMOE_ERR_INVALID_ARG;

  unsigned char* base = nullptr;
  if (scratch_address(&base) != cudaSuccess) return CMOE_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  float* Ct = reinterpret_cast<float*>(base + off_ct);
  float* Rt = reinterpret_cast<float*>(base + off_rt);
  float* bc = reinterpret_cast<float*>(base + off_bc);
  float* be = reinterpret_cast<float*>(base + off_be);
  int* label = reinterpret_cast<int*>(base + off_lb);

  cudaError_t e;
  if ((e = launch_transpose_f32(C, Ct, 1, d, G, st)) != cudaSuccess) return CMOE_ERR_CUDA;
  if ((e = launch_transpose_f32(R, Rt, G, d, K, st)) != cudaSuccess) return CMOE_ERR_CUDA;
  // the array still holds the previous call's biases: overwrite them, with zeros if none are given
  e = b_c ? cudaMemcpyAsync(bc, b_c, sizeof(float) * (size_t)G, cudaMemcpyDeviceToDevice, st)
          : cudaMemsetAsync(bc, 0, sizeof(float) * (size_t)G, st);
  if (e != cudaSuccess) return CMOE_ERR_CUDA;
  e = b_e ? cudaMemcpyAsync(be, b_e, sizeof(float) * (size_t)E, cudaMemcpyDeviceToDevice, st)
          : cudaMemsetAsync(be, 0, sizeof(float) * (size_t)E, st);
  if (e != cudaSuccess) return CMOE_ERR_CUDA;
  iota_kernel<<<(E + 127) / 128, 128, 0, st>>>(label, E);
  if ((e = cudaGetLastError()) != cudaSuccess) return CMOE_ERR_CUDA;

  Dims D{};
  D.d = d; D.E = E; D.G = G; D.K = K; D.k = k;
  Weights W{};
  W.Ct = Ct; W.Rt = Rt; W.bc = bc; W.be = be; W.label = label;
  if (launch_router(D, W, static_cast<const __half*>(x), T, cluster_id, expert_ids, gates, nullptr,
                    st) != cudaSuccess)
    return CMOE_ERR_CUDA;
  return CMOE_OK;
}
