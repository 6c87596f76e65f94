// sdgp_dgrad_linear_static: the two-pass fully connected data gradient for callers that
// cannot hand the library a workspace because they cannot allocate device memory at the
// point of the call - code running inside another framework's allocator-free region, a
// plugin whose host forbids cudaMalloc after start-up, or a real-time loop where an
// allocation's implicit synchronisation is not acceptable. The scratch that
// sdgp_dgrad_linear takes from its `workspace` argument lives here in a fixed array in
// device global memory instead.
#include "sdgp_internal.cuh"

namespace {

// Compressed dL/dO of one call: rows*K bytes of values followed (256-byte aligned) by
// rows*K/8 bytes of position metadata. 9 MiB on every GPU that loads the library, until exit.
constexpr size_t kMaxElements = (size_t)8 << 20;  // rows * K
constexpr size_t kValuesBytes = kMaxElements;
constexpr size_t kMetaBytes = kMaxElements / 8;
static __device__ __align__(256) unsigned char g_static_scratch[kValuesBytes + kMetaBytes];

constexpr int kMaxDevices = 64;
unsigned char* g_scratch_addr[kMaxDevices] = {};

// In host code `g_static_scratch` is only a handle for the symbol, not a device address;
// the address the kernels need is asked for once per device, with that device current.
// Threads that make their first call on a device at the same time may each do the lookup; they
// all store the same address, so no lock is taken.
sdgp_status scratch_for_current_device(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SDGP_ERR_CUDA;
  if (!g_scratch_addr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return SDGP_ERR_CUDA;
    g_scratch_addr[dev] = (unsigned char*)ptr;
  }
  *out = g_scratch_addr[dev];
  return SDGP_OK;
}

}  // namespace

extern "C" sdgp_status sdgp_dgrad_linear_static(const void* dO, const void* W, void* dD, int64_t rows,
                                                 int64_t K, int64_t N, int n, int m, sdgp_scheme scheme,
                                                 uint64_t seed, void* stream) {
  if (rows < 0 || K < 1 || N < 1) return SDGP_ERR_INVALID_ARG;
  if ((int)scheme < 0 || (int)scheme > 2) return SDGP_ERR_INVALID_ARG;
  if (m < 1 || m > 32 || n < 1 || n > m) return SDGP_ERR_INVALID_ARG;
  if (m != 4 && m != 8 && m != 16 && m != 32) return SDGP_ERR_UNSUPPORTED;
  if (K % m != 0) return SDGP_ERR_INVALID_ARG;
  if (n > 2 && n != m) return SDGP_ERR_UNSUPPORTED;
  if (K % 128 != 0 || N % 64 != 0) return SDGP_ERR_UNSUPPORTED;
  if (rows > 0x7FFFFFFF || K > 0x7FFFFFFF || N > 0x7FFFFFFF) return SDGP_ERR_UNSUPPORTED;
  if ((uint64_t)rows * (uint64_t)K > kMaxElements) return SDGP_ERR_TOO_LARGE;
  if (rows == 0) return SDGP_OK;
  if (!dO || !W || !dD) return SDGP_ERR_INVALID_ARG;
  if (((uintptr_t)dO | (uintptr_t)W | (uintptr_t)dD) & 15u) return SDGP_ERR_ALIGNMENT;
  cudaStream_t s = (cudaStream_t)stream;
  // n == m prunes nothing: the dense kernel reads dO itself and the scratch is not touched
  if (n == m) return sdgp::launch_dgrad(false, dO, nullptr, W, dD, 1, 1, (int)rows, (int)N, (int)K, 1, 1, 1, 0, s);

  unsigned char* scratch = nullptr;
  sdgp_status st = scratch_for_current_device(&scratch);
  if (st != SDGP_OK) return st;
  void* values = scratch;
  void* meta = scratch + kValuesBytes;
  // Every byte of values/meta that the contraction reads is rewritten by the prune kernel
  // first, so what an earlier call left in the array never shows.
  if (sdgp::launch_prune(dO, rows, K, n, m, (int)scheme, seed, nullptr, values, meta, nullptr, s) != cudaSuccess)
    return SDGP_ERR_CUDA;
  return sdgp::launch_dgrad(true, values, meta, W, dD, 1, 1, (int)rows, (int)N, (int)K, 1, 1, 1, 0, s);
}
