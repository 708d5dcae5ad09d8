// Launch-layer interface between the C ABI (aq_api.cu) and the kernels (aq_kernels.cu, aq_lowbit.cu).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace aq {

constexpr int kChunk = 8;            // elements per 128-bit access of a 2-byte type
constexpr int kThreads = 256;        // threads per CTA; one "row" = kThreads consecutive chunks
constexpr int kRowsPerIter = 2;      // rows a CTA has in flight per loop iteration
constexpr int kMaxBatch = 4096;      // samples per encode / decode call

// "Seen before" is kept as a stamp per sample: 0 = never seen, otherwise the number of the
// call that saw it first (kImportedStamp for a sample loaded through aq_import_sample).  A
// sample whose stamp equals the number of the running call is still a first visit for every
// CTA of that call, so the stamp may be written while other CTAs are reading it.
constexpr unsigned long long kImportedStamp = 1ull;
constexpr unsigned long long kFirstCall = 2ull;
// what one encode / decode launch adds to the handle's arrival counter; also the largest grid
constexpr unsigned long long kCallQuantum = 1ull << 20;

// State of one side of a boundary, as the kernels see it.
struct State {
  void* m;                        // T[n_samples][elems]; low-precision store: uint8[n_samples][m_bytes] codes
  float* m_scales;                // low-precision store: float[n_samples][groups] steps of m; else null
  long long m_bytes;              // low-precision store: bytes of codes per sample (elems * m_bits / 8)
  int m_bits;                     // 0: m kept in the activation type; 2, 4, 8: low-precision store
  unsigned long long* seen;       // [n_samples] stamps
  unsigned long long* arrivals;   // grows by kCallQuantum per encode / decode launch (starts at 0)
  uint32_t* status;               // sticky AQ_ST_* bits
  long long n_samples;
  long long elems;                // seq * hidden
  long long packed_bytes;         // per sample
  long long groups;               // per sample
  int chunks;                     // elems / 8
  int rows;                       // ceil(chunks / kThreads): rows per sample
  int lanes_per_group;            // group / 8: a power of two <= 32 for the kernels of aq_kernels.cu and aq_lowbit.cu
  int lg_shift;                   // log2(lanes_per_group); -1: any other lane count (kernels of aq_anygroup.cu)
  int sms;                        // multiprocessors of the handle's device
  int rows_per_cta;               // 0 = chosen by the launch layer (default); > 0 = fixed rows per CTA
  int l2_prefetch;                // 1: encode / decode ask for a CTA's rows to be brought into L2 ahead of its loads
  const int32_t* slot_ids;        // null: row xi of m belongs to sample xi.  Else m is a staging block of the
                                  // running call: row y holds m of sample slot_ids[y] (hosted store, prefetched)
};

// A call names its buffers either by one base pointer each (sample y at base + y * its size) or,
// when `lists` is set, by device arrays of n_batch pointers, one buffer per sample.
struct EncodeArgs {
  const void* act;
  const int32_t* ids;
  uint8_t* packed;
  float* scales;
  uint8_t* first_flags;    // may be null
  int n_batch;
  bool stochastic;                  // unbiased stochastic rounding instead of the interval number
  unsigned long long seed, epoch;   // its generator key and the caller's call counter
  bool lists;                       // act, packed, scales are arrays of pointers (act_list() etc.)
  __host__ __device__ const void* const* act_list() const { return static_cast<const void* const*>(act); }
  __host__ __device__ const void* const* packed_list() const { return reinterpret_cast<const void* const*>(packed); }
  __host__ __device__ const void* const* scales_list() const { return reinterpret_cast<const void* const*>(scales); }
};

struct DecodeArgs {
  const uint8_t* packed;
  const float* scales;
  const void* raw;         // may be null (as a list: the array itself, or single entries of it)
  const int32_t* ids;
  void* out;
  uint8_t* first_flags;    // may be null
  int n_batch;
  bool lists;              // packed, scales, raw, out are arrays of pointers
  __host__ __device__ const void* const* packed_list() const { return reinterpret_cast<const void* const*>(packed); }
  __host__ __device__ const void* const* scales_list() const { return reinterpret_cast<const void* const*>(scales); }
  __host__ __device__ const void* const* raw_list() const { return static_cast<const void* const*>(raw); }
  __host__ __device__ const void* const* out_list() const { return static_cast<const void* const*>(out); }
};

cudaError_t launch_encode(int dtype, int bits, const State& st, const EncodeArgs& a, cudaStream_t s);
cudaError_t launch_decode(int dtype, int bits, const State& st, const DecodeArgs& a, cudaStream_t s);
cudaError_t launch_encode_lowbit(int dtype, int bits, const State& st, const EncodeArgs& a, cudaStream_t s);
cudaError_t launch_decode_lowbit(int dtype, int bits, const State& st, const DecodeArgs& a, cudaStream_t s);
cudaError_t launch_quant_grad(int dtype, int bits, int lanes_per_group, const void* grad,
                              long long n_elems, uint8_t* packed, float* scales, bool stochastic,
                              unsigned long long seed, unsigned long long epoch, int l2_prefetch, cudaStream_t s);
cudaError_t launch_dequant_grad(int dtype, int bits, int lanes_per_group, const uint8_t* packed,
                                const float* scales, long long n_elems, void* out, cudaStream_t s);
// The same four for groups whose lane count is not a power of two up to 32 (aq_anygroup.cu; 16-bit store).
cudaError_t launch_encode_anygroup(int dtype, int bits, const State& st, const EncodeArgs& a, cudaStream_t s);
cudaError_t launch_decode_anygroup(int dtype, int bits, const State& st, const DecodeArgs& a, cudaStream_t s);
cudaError_t launch_quant_grad_anygroup(int dtype, int bits, int lanes_per_group, const void* grad, long long n_elems,
                                       uint8_t* packed, float* scales, bool stochastic, unsigned long long seed,
                                       unsigned long long epoch, cudaStream_t s);
cudaError_t launch_dequant_grad_anygroup(int dtype, int bits, int lanes_per_group, const uint8_t* packed, const float* scales,
                                         long long n_elems, void* out, cudaStream_t s);
// Rows of `row_bytes` bytes moved by one kernel (in 16-, 4- or 1-byte pieces, as the size and the bases allow): gather: dst row y <- src row
// ids[y]; scatter: dst row ids[y] <- src row y; entries with ids[y] < 0 are left out.
cudaError_t launch_copy_rows(const void* src, void* dst, const int32_t* ids, int n, long long row_bytes, bool gather,
                             cudaStream_t s);
// Up to three byte ranges (sizes multiples of 16, bases 16-byte aligned, all on the current device) copied by
// one kernel launch.
cudaError_t launch_wire_copy(const void* const* src, void* const* dst, const size_t* bytes, int n_ranges, cudaStream_t s);
// *sum_dev += digest of (m, seen); the caller zeroes *sum_dev first.
cudaError_t launch_checksum(const State& st, unsigned long long* sum_dev, cudaStream_t s);

}  // namespace aq

// The handle is defined in aq_api.cu; entry points in other files reach it through these.
struct aq_handle;
namespace aq {
const State* handle_state(aq_handle* h);
cudaStream_t handle_stream(aq_handle* h);
int handle_device(aq_handle* h);
int handle_fail(aq_handle* h, int code, const char* msg);   // records msg for aq_last_error, returns code
cudaError_t handle_settle(aq_handle* h);   // hosted store: makes the handle's stream wait for write-backs in flight
}  // namespace aq
