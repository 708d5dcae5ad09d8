// aq_state_checksum_noalloc: the state digest for callers that must not allocate.
//
// Who needs it: code that runs where device allocation is off limits -- a process whose device
// memory was all handed out at start-up (a caching pool owns it; a cudaMalloc from a library would
// fail or force the pool to give memory back), a step loop that may not take the device-wide
// synchronisation cudaMalloc and cudaFree can bring, a service that gives every library a fixed
// memory budget.  Such a caller cannot give this library a chance to cudaMalloc its working
// memory, so the working memory of this entry point is part of the library image: a fixed array
// in device memory that every GPU holds from the moment the library is loaded on it until the
// process exits.  The call still synchronises the handle's stream and returns the digest in host
// memory, exactly like aq_state_checksum.
//
// The digest is the one aq_state_checksum returns.  It is formed in two steps: every CTA sums
// the mixed words of one slab of m into its own slot of the fixed array, then one CTA adds the
// slots and the terms of the seen-set.  The number of slots bounds the size of m that one call
// can digest (kSlots slabs of 1 MiB).

#include "../../include/aq_b200.h"
#include "aq_internal.h"

#include <mutex>

namespace {

constexpr int kSlabVecs = 1 << 16;                         // 16-byte pieces of m per CTA: 1 MiB
constexpr int kSlots = 1 << 16;                            // partial sums: up to 64 GiB of m per call
constexpr int kMaxDevices = 64;

// kSlots partial sums and, after them, the finished digest.  512 KiB + 256 B on every GPU that
// loads the library.  Shared by all calls: it keeps what the last call left, every call
// rewrites each slot it reads, and two calls that overlap on one GPU race on it.
static __device__ __align__(256) unsigned long long g_digest_scratch[kSlots + 32];

__device__ __forceinline__ unsigned long long mix64(unsigned long long index, unsigned long long word) {
  unsigned long long z = index * 0x9E3779B97F4A7C15ull + word;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

__device__ __forceinline__ unsigned long long cta_sum(unsigned long long acc, unsigned long long* part) {
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
  __syncthreads();
  unsigned long long t = 0ull;
  if (threadIdx.x == 0)
    for (int w = 0; w < aq::kThreads / 32; ++w) t += part[w];
  return t;                                                // valid in thread 0
}

// slot[b] = sum of mix(i, word_i) over the words of slab b of m
__global__ void __launch_bounds__(aq::kThreads) digest_slabs_kernel(const uint4* __restrict__ mv, long long n_vec,
                                                                     unsigned long long* __restrict__ slot) {
  __shared__ unsigned long long part[aq::kThreads / 32];
  const long long v0 = (long long)blockIdx.x * kSlabVecs;
  const long long v1 = (v0 + kSlabVecs < n_vec) ? v0 + kSlabVecs : n_vec;
  unsigned long long acc = 0ull;
  for (long long v = v0 + threadIdx.x; v < v1; v += aq::kThreads) {
    const uint4 w = __ldcs(mv + v);
    const unsigned long long i = (unsigned long long)v * 2ull;           // two 64-bit words per piece
    acc += mix64(i, ((unsigned long long)w.y << 32) | w.x) + mix64(i + 1, ((unsigned long long)w.w << 32) | w.z);
  }
  const unsigned long long t = cta_sum(acc, part);
  if (threadIdx.x == 0) slot[blockIdx.x] = t;
}

// slot[kSlots] = sum of the n_slots partial sums + the seen-set terms
__global__ void __launch_bounds__(aq::kThreads) digest_finish_kernel(const unsigned long long* __restrict__ seen,
                                                                      long long n_samples, int n_slots,
                                                                      unsigned long long* __restrict__ slot) {
  __shared__ unsigned long long part[aq::kThreads / 32];
  unsigned long long acc = 0ull;
  for (int b = threadIdx.x; b < n_slots; b += aq::kThreads) acc += slot[b];
  for (long long x = threadIdx.x; x < n_samples; x += aq::kThreads)
    acc += mix64((1ull << 40) + (unsigned long long)x, seen[x] != 0ull ? 1ull : 0ull);
  const unsigned long long t = cta_sum(acc, part);
  if (threadIdx.x == 0) slot[kSlots] = t;
}

// Device address of the fixed array on `device` (which must be current).  In host code the
// array's name is only a handle for the runtime; the address a kernel can use has to be asked
// for, once per device.  The first call of the entry point on a device does this and should come
// before any stream capture begins; the address is kept until the process ends (a cudaDeviceReset
// would make it stale).
std::mutex g_setup_lock;
unsigned long long* g_scratch_addr[kMaxDevices] = {nullptr};

cudaError_t scratch_address(int device, unsigned long long** out) {
  std::lock_guard<std::mutex> hold(g_setup_lock);
  if (!g_scratch_addr[device]) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_digest_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_addr[device] = static_cast<unsigned long long*>(p);
  }
  *out = g_scratch_addr[device];
  return cudaSuccess;
}

}  // namespace

extern "C" int aq_state_checksum_noalloc(aq_handle* h, uint64_t* out_host) {
  if (!h) return AQ_EINVAL;
  if (!out_host) return aq::handle_fail(h, AQ_EINVAL, "aq_state_checksum_noalloc: null pointer");
  const aq::State& st = *aq::handle_state(h);
  if (st.m_bits)
    return aq::handle_fail(h, AQ_EUNSUPPORTED, "aq_state_checksum_noalloc: not built for the low-precision and binary32 stores");
  const long long n_vec = st.n_samples * (long long)st.chunks;
  const long long n_slots = (n_vec + kSlabVecs - 1) / kSlabVecs;
  if (n_slots > kSlots)
    return aq::handle_fail(h, AQ_EUNSUPPORTED,
                           "aq_state_checksum_noalloc: m is larger than the 64 GiB that the fixed scratch array covers");
  const int device = aq::handle_device(h);
  if (device < 0 || device >= kMaxDevices)
    return aq::handle_fail(h, AQ_EUNSUPPORTED, "aq_state_checksum_noalloc: device index beyond 63");
  int prev = -1;
  cudaGetDevice(&prev);
  if (prev != device) cudaSetDevice(device);
  unsigned long long* scratch = nullptr;
  cudaError_t e = scratch_address(device, &scratch);
  const cudaStream_t stream = aq::handle_stream(h);
  unsigned long long v = 0;
  if (e == cudaSuccess) e = aq::handle_settle(h);
  if (e == cudaSuccess) {
    digest_slabs_kernel<<<(unsigned)n_slots, aq::kThreads, 0, stream>>>(static_cast<const uint4*>(st.m), n_vec, scratch);
    digest_finish_kernel<<<1, aq::kThreads, 0, stream>>>(st.seen, st.n_samples, (int)n_slots, scratch);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(&v, scratch + kSlots, sizeof(v), cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  if (prev != device && prev >= 0) cudaSetDevice(prev);
  if (e != cudaSuccess) return aq::handle_fail(h, AQ_ECUDA, cudaGetErrorString(e));
  *out_host = v;
  return AQ_OK;
}
