// percache_debug_gemm_noalloc: the GEMM test hook for callers that must not allocate device memory.
//
// Who needs it: a process that has already handed the whole GPU to another allocator (a framework's
// caching pool sized to all of device memory), where a raw cudaMalloc simply fails; and a serving loop
// that cannot afford the device-wide synchronisation cudaMalloc / cudaFree imply.  For them the device
// copies of A, B, C and the kernel's error word live in a fixed array that is part of the library
// image: every GPU that loads the library holds NOALLOC_SCRATCH_BYTES of it until the process exits.
#include <cstring>

#include "../../include/percache.h"
#include "kernels.h"

using namespace pc;

namespace {

constexpr size_t NOALLOC_SCRATCH_BYTES = PERCACHE_NOALLOC_SCRATCH_BYTES;
constexpr int MAX_DEVICES = 64;

// The scratch itself.  In host code this name is only a handle for the runtime, not a device
// address: the address a kernel may use comes from cudaGetSymbolAddress (below), once per device.
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_SCRATCH_BYTES];

unsigned char* g_scratch_addr[MAX_DEVICES] = {};

size_t round256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

// Device address of the scratch on `device` (which must be current).  Looked up on the first call for
// that device and remembered.
int scratch_address(int device, unsigned char** out) {
  if (device < 0 || device >= MAX_DEVICES) return PERCACHE_E_INVAL;
  if (!g_scratch_addr[device]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return PERCACHE_E_CUDA;
    }
    g_scratch_addr[device] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_addr[device];
  return PERCACHE_OK;
}

}  // namespace

extern "C" int percache_debug_gemm_noalloc(int32_t device, int32_t M, int32_t N, int32_t K, const void* a_f16,
                                           const void* b_f16, float* c) {
  if (M <= 0 || N <= 0 || K <= 0 || !a_f16 || !b_f16 || !c) return PERCACHE_E_INVAL;
  if (K % 64 != 0 || N % 128 != 0) return PERCACHE_E_INVAL;
  // layout of the scratch: [error word | A padded to whole 128-row tiles | B | C], each 256-byte aligned
  const size_t m_pad = (static_cast<size_t>(M) + 127) / 128 * 128;     // in size_t: M may be close to INT32_MAX
  const size_t a_bytes = round256(m_pad * K * 2), b_bytes = round256(static_cast<size_t>(N) * K * 2);
  const size_t c_bytes = round256(static_cast<size_t>(M) * N * 4);
  if (256 + a_bytes + b_bytes + c_bytes > NOALLOC_SCRATCH_BYTES) return PERCACHE_E_CAPACITY;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device < 0 || device >= n_dev) { cudaGetLastError(); return PERCACHE_E_CUDA; }
  if (cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return PERCACHE_E_CUDA; }
  if (init_driver_api() != 0) return PERCACHE_E_CUDA;
  unsigned char* base = nullptr;
  int rc = scratch_address(device, &base);
  if (rc != PERCACHE_OK) return rc;
  int* d_err = reinterpret_cast<int*>(base);
  __half* dA = reinterpret_cast<__half*>(base + 256);
  __half* dB = reinterpret_cast<__half*>(base + 256 + a_bytes);
  float* dC = reinterpret_cast<float*>(base + 256 + a_bytes + b_bytes);
  // The array keeps whatever the previous call left: clear the error word and the padding rows of A.
  bool ok = cudaMemset(d_err, 0, 256) == cudaSuccess;
  if (m_pad > static_cast<size_t>(M))
    ok = ok && cudaMemset(dA + static_cast<size_t>(M) * K, 0, (m_pad - M) * K * 2) == cudaSuccess;
  ok = ok && cudaMemcpy(dA, a_f16, static_cast<size_t>(M) * K * 2, cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(dB, b_f16, static_cast<size_t>(N) * K * 2, cudaMemcpyHostToDevice) == cudaSuccess;
  GemmOperand mA, mB;
  int n_sms = 148;
  cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, device);
  ok = ok && make_operand_map(&mA, dA, static_cast<int64_t>(m_pad), K, 128) == 0 &&
       make_operand_map(&mB, dB, N, K, 128) == 0 &&
       launch_umma_gemm(mA, mB, M, N, K, 128, EPI_STORE_F32, nullptr, dC, d_err, n_sms, nullptr) == 0;
  if (!ok || cudaDeviceSynchronize() != cudaSuccess || cudaGetLastError() != cudaSuccess) {
    cudaGetLastError();
    return PERCACHE_E_CUDA;
  }
  int h_err = 0;
  if (cudaMemcpy(&h_err, d_err, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return PERCACHE_E_CUDA;
  if (h_err != 0) return PERCACHE_E_DEVICE_TIMEOUT;
  if (cudaMemcpy(c, dC, static_cast<size_t>(M) * N * 4, cudaMemcpyDeviceToHost) != cudaSuccess) return PERCACHE_E_CUDA;
  return PERCACHE_OK;
}
