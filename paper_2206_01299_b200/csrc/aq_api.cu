// C ABI of the codec: handle, argument checks, stream plumbing.  All arithmetic lives in
// aq_kernels.cu and aq_lowbit.cu; nothing here computes on the CPU and there is no CPU fallback.

#include "../../include/aq_b200.h"
#include "aq_internal.h"

#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <unordered_set>
#include <vector>

struct aq_handle {
  aq::State st{};
  int seq = 0, hidden = 0, bits = 0, group = 0;
  int dtype = AQ_FP16;
  int n_batch = 1;
  int l2_prefetch = 1;                       // AQ_L2_PREFETCH as set; st.l2_prefetch is what in-place calls get
  int rounding = AQ_ROUND_INTERVAL;
  unsigned long long seed = 0, epoch = 0;
  int device = 0;
  cudaStream_t stream = nullptr;
  const void* raw = nullptr;
  const void* const* raw_list = nullptr;     // AQ_RAW_LIST: the raw messages of a list-form decode
  uint8_t* first_flags = nullptr;
  unsigned long long* sum_dev = nullptr;     // scratch of aq_state_checksum
  void* m_host = nullptr;                    // hosted store: the pinned host block that st.m maps
  float* m_scales_host = nullptr;            // ... and the one that st.m_scales maps (low-precision hosted store)
  // hosted store, staged visits: aq_prefetch copies the next call's m(xi) into a staging block in device
  // memory on fetch_stream, the call works there and copies the rows back on store_stream afterwards.  Two
  // blocks are used in turn, so that the rows of call N+1 arrive while call N computes and while its rows
  // travel home, and the two directions of the host link work at the same time.
  struct Stage {
    void* slots = nullptr;                   // [batch] rows of m (16-bit values, or the codes of a low-precision store)
    float* slot_scales = nullptr;            // [batch][groups] steps of those rows (low-precision store)
    int32_t* d_slot_ids = nullptr;           // [batch] ids as given to aq_prefetch
    int32_t* d_copy_ids = nullptr;           // [batch] the same with -1 where no row is to be moved
    int batch = 0;
    std::vector<int32_t> ids;                // per slot: the sample whose row it holds, -1 = nothing to copy
    bool rows_by_kernel = false;             // how this block's rows travel (see aq_prefetch)
    cudaEvent_t ev_staged = nullptr;         // fetch_stream: the prefetched rows are in HBM
    cudaEvent_t ev_computed = nullptr;       // the handle's stream: the call that used them is done
    cudaEvent_t ev_written = nullptr;        // store_stream: its rows are back in host memory
    bool writeback_issued = false;
  };
  static constexpr int kStages = 2;
  Stage stage[kStages];
  int next_stage = 0;                        // the block that the next aq_prefetch fills
  int pending_stage = -1;                    // the block of the pending prefetch, -1 = none
  cudaStream_t fetch_stream = nullptr, store_stream = nullptr;
  cudaEvent_t ev_settled = nullptr;          // the handle's stream, when aq_prefetch was called
  // the ids travel to d_slot_ids from page-locked blocks used in turn (a pageable source would
  // make the copy wait on the host for fetch_stream to drain); an event says when one is free again
  static constexpr int kIdRing = 4;
  int32_t* ids_pinned[kIdRing] = {nullptr, nullptr, nullptr, nullptr};
  cudaEvent_t ev_ids_sent[kIdRing] = {nullptr, nullptr, nullptr, nullptr};
  unsigned prefetches = 0;
  bool inplace_since_fetch = true;           // a call worked on the host block in place since the last prefetch was issued
  // staging for the host-buffer entry points, sized for staged_batch samples
  int staged_batch = 0;
  void* d_act = nullptr;      // also raw / out
  int32_t* d_ids = nullptr;
  uint8_t* d_packed = nullptr;
  float* d_scales = nullptr;
  // the host-buffer calls move a batch in kSlices pieces: copies in on in_stream, kernels on the
  // handle's stream, copies out on out_stream, so that neighbouring pieces overlap
  static constexpr int kSlices = 4;
  cudaStream_t in_stream = nullptr, out_stream = nullptr;
  cudaEvent_t ev_begin = nullptr, ev_in[kSlices] = {}, ev_done[kSlices] = {};
  char err[256] = {0};
  int err_code = AQ_OK;                      // code of the call that wrote err
};

namespace {

thread_local char g_create_err[256] = "";
thread_local int g_create_code = AQ_OK;

int fail(aq_handle* h, int code, const char* fmt, ...) {
  char* dst = h ? h->err : g_create_err;
  (h ? h->err_code : g_create_code) = code;
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(dst, 256, fmt, ap);
  va_end(ap);
  return code;
}

int cuda_fail(aq_handle* h, cudaError_t e, const char* what) {
  return fail(h, e == cudaErrorMemoryAllocation ? AQ_ENOMEM : AQ_ECUDA, "%s: %s", what, cudaGetErrorString(e));
}

#define AQ_CUDA(h, call)                                   \
  do {                                                     \
    cudaError_t e_ = (call);                               \
    if (e_ != cudaSuccess) return cuda_fail(h, e_, #call); \
  } while (0)

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int lanes_for_group(int group) {
  switch (group) {
    case 8: case 16: case 32: case 64: case 128: case 256: return group / 8;
    default: return 0;
  }
}

// The handle's device must be current for launches on its stream; restore on exit.
struct DeviceGuard {
  int prev = -1;
  explicit DeviceGuard(int dev) {
    cudaGetDevice(&prev);
    if (prev != dev) cudaSetDevice(dev);
    else prev = -1;
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

void free_staging(aq_handle* h) {
  cudaFree(h->d_act); cudaFree(h->d_ids); cudaFree(h->d_packed); cudaFree(h->d_scales);
  h->d_act = nullptr; h->d_ids = nullptr; h->d_packed = nullptr; h->d_scales = nullptr;
  h->staged_batch = 0;
}

int ensure_staging(aq_handle* h) {
  if (h->staged_batch >= h->n_batch && h->d_act) return AQ_OK;
  AQ_CUDA(h, cudaStreamSynchronize(h->stream));
  free_staging(h);
  const size_t nb = (size_t)(h->n_batch > 0 ? h->n_batch : 1);
  AQ_CUDA(h, cudaMalloc(&h->d_act, nb * (size_t)h->st.elems * 2));
  AQ_CUDA(h, cudaMalloc(reinterpret_cast<void**>(&h->d_ids), nb * sizeof(int32_t)));
  AQ_CUDA(h, cudaMalloc(reinterpret_cast<void**>(&h->d_packed), nb * (size_t)h->st.packed_bytes));
  AQ_CUDA(h, cudaMalloc(reinterpret_cast<void**>(&h->d_scales), nb * (size_t)h->st.groups * sizeof(float)));
  h->staged_batch = (int)nb;
  return AQ_OK;
}

int ensure_slicing(aq_handle* h) {
  if (h->in_stream) return AQ_OK;
  AQ_CUDA(h, cudaStreamCreateWithFlags(&h->in_stream, cudaStreamNonBlocking));
  AQ_CUDA(h, cudaStreamCreateWithFlags(&h->out_stream, cudaStreamNonBlocking));
  AQ_CUDA(h, cudaEventCreateWithFlags(&h->ev_begin, cudaEventDisableTiming));
  for (int i = 0; i < aq_handle::kSlices; ++i) {
    AQ_CUDA(h, cudaEventCreateWithFlags(&h->ev_in[i], cudaEventDisableTiming));
    AQ_CUDA(h, cudaEventCreateWithFlags(&h->ev_done[i], cudaEventDisableTiming));
  }
  return AQ_OK;
}

// A host-buffer call may run in slices when every id is in range and appears once (the kernels
// look for repeats inside one launch only) and m is in device memory.
bool sliceable(const aq_handle* h, const int32_t* ids_host) {
  if (h->n_batch < 2 * aq_handle::kSlices || h->m_host) return false;
  std::unordered_set<int32_t> taken;
  for (int j = 0; j < h->n_batch; ++j) {
    const int32_t id = ids_host[j];
    if (id < 0 || (long long)id >= h->st.n_samples || !taken.insert(id).second) return false;
  }
  return true;
}

// Hosted store: rows that staged calls updated travel back to host memory on store_stream.
// Whatever touches the host block next on the handle's stream waits for them on the device.
cudaError_t settle(aq_handle* h) {
  for (aq_handle::Stage& sg : h->stage) {
    if (!sg.writeback_issued) continue;
    const cudaError_t e = cudaStreamWaitEvent(h->stream, sg.ev_written, 0);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// The rows of one staging block between the host blocks and the block, on `stream`: in = host to
// staging.  A low-precision store has two blocks, codes and steps.
int move_rows(aq_handle* h, aq_handle::Stage& sg, bool in, cudaStream_t stream) {
  const int n = (int)sg.ids.size();
  const size_t bytes = (size_t)h->st.m_bytes, step_bytes = (size_t)h->st.groups * sizeof(float);
  const cudaMemcpyKind kind = in ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToHost;
  if (sg.rows_by_kernel) {
    AQ_CUDA(h, aq::launch_copy_rows(in ? h->st.m : sg.slots, in ? sg.slots : h->st.m, sg.d_copy_ids, n, (long long)bytes, in, stream));
    if (h->m_scales_host)
      AQ_CUDA(h, aq::launch_copy_rows(in ? h->st.m_scales : sg.slot_scales, in ? sg.slot_scales : h->st.m_scales, sg.d_copy_ids,
                                      n, (long long)step_bytes, in, stream));
    return AQ_OK;
  }
  for (int j = 0; j < n; ++j) {
    const int32_t id = sg.ids[j];
    if (id < 0) continue;
    char* host_row = static_cast<char*>(h->m_host) + (size_t)id * bytes;
    char* slot_row = static_cast<char*>(sg.slots) + (size_t)j * bytes;
    AQ_CUDA(h, cudaMemcpyAsync(in ? slot_row : host_row, in ? host_row : slot_row, bytes, kind, stream));
    if (h->m_scales_host) {
      float* host_steps = h->m_scales_host + (size_t)id * (size_t)h->st.groups;
      float* slot_steps = sg.slot_scales + (size_t)j * (size_t)h->st.groups;
      AQ_CUDA(h, cudaMemcpyAsync(in ? slot_steps : host_steps, in ? host_steps : slot_steps, step_bytes, kind, stream));
    }
  }
  return AQ_OK;
}

// A staged call: `launch` runs on the prefetched rows in HBM, then the rows go home on store_stream.
template <typename Launch>
int run_staged(aq_handle* h, Launch launch) {
  aq_handle::Stage& sg = h->stage[h->pending_stage];
  h->pending_stage = -1;
  if ((int)sg.ids.size() != h->n_batch)
    return fail(h, AQ_EINVAL, "the pending aq_prefetch was for %d samples, AQ_BATCH is %d", (int)sg.ids.size(), h->n_batch);
  aq::State st = h->st;
  st.m = sg.slots;
  if (h->m_scales_host) st.m_scales = sg.slot_scales;
  st.slot_ids = sg.d_slot_ids;
  st.l2_prefetch = h->l2_prefetch;                    // the staged rows are in device memory
  AQ_CUDA(h, cudaStreamWaitEvent(h->stream, sg.ev_staged, 0));
  AQ_CUDA(h, launch(st));
  AQ_CUDA(h, cudaEventRecord(sg.ev_computed, h->stream));
  AQ_CUDA(h, cudaStreamWaitEvent(h->store_stream, sg.ev_computed, 0));
  const int rc = move_rows(h, sg, false, h->store_stream);
  if (rc != AQ_OK) return rc;
  AQ_CUDA(h, cudaEventRecord(sg.ev_written, h->store_stream));
  sg.writeback_issued = true;
  return AQ_OK;
}

}  // namespace

extern "C" {

static aq_handle* create_handle(int64_t n_samples, int seq, int hidden, int bits, int group, int m_bits,
                                bool hosted = false);

aq_handle* aq_create(int64_t n_samples, int seq, int hidden, int bits, int group) {
  return create_handle(n_samples, seq, hidden, bits, group, 0);
}

aq_handle* aq_create_hosted(int64_t n_samples, int seq, int hidden, int bits, int group) {
  return create_handle(n_samples, seq, hidden, bits, group, 0, true);
}

aq_handle* aq_create_hosted_lowbit(int64_t n_samples, int seq, int hidden, int bits, int group, int m_bits) {
  if (m_bits != 2 && m_bits != 4 && m_bits != 8) {
    g_create_err[0] = 0;
    fail(nullptr, AQ_EINVAL, "m_bits must be 2, 4 or 8 (got %d)", m_bits);
    return nullptr;
  }
  return create_handle(n_samples, seq, hidden, bits, group, m_bits, true);
}

aq_handle* aq_create_fp32(int64_t n_samples, int seq, int hidden, int bits, int group) {
  return create_handle(n_samples, seq, hidden, bits, group, 32);
}

aq_handle* aq_create_lowbit(int64_t n_samples, int seq, int hidden, int bits, int group, int m_bits) {
  if (m_bits != 2 && m_bits != 4 && m_bits != 8) {
    g_create_err[0] = 0;
    fail(nullptr, AQ_EINVAL, "m_bits must be 2, 4 or 8 (got %d)", m_bits);
    return nullptr;
  }
  return create_handle(n_samples, seq, hidden, bits, group, m_bits);
}

static aq_handle* create_handle(int64_t n_samples, int seq, int hidden, int bits, int group, int m_bits,
                                bool hosted) {
  g_create_err[0] = 0;
  g_create_code = AQ_OK;
  const int lanes = lanes_for_group(group);
  if (n_samples <= 0 || seq <= 0 || hidden <= 0) { fail(nullptr, AQ_EINVAL, "n_samples, seq and hidden must be positive"); return nullptr; }
  if (n_samples > 0x7fffffffll) { fail(nullptr, AQ_EINVAL, "n_samples must fit the int32 sample ids"); return nullptr; }
  if ((long long)seq * hidden > (1ll << 30)) { fail(nullptr, AQ_EINVAL, "seq*hidden must not exceed 2^30 elements per sample"); return nullptr; }
  if (bits < 1 || bits > 8) { fail(nullptr, AQ_EINVAL, "bits must be in 1..8 (got %d)", bits); return nullptr; }
  if (group <= 0 || group % 8) { fail(nullptr, AQ_EINVAL, "group must be a positive multiple of 8 (got %d)", group); return nullptr; }
  if (hidden % group) { fail(nullptr, AQ_EINVAL, "group %d does not divide hidden %d", group, hidden); return nullptr; }
  if (!lanes && m_bits) {
    // a valid quantizer setting that the kernels of the low-precision and binary32 stores are not built for:
    // there the lanes that share a group's maximum must be a power of two within one warp
    fail(nullptr, AQ_EUNSUPPORTED, "group %d: the low-precision and binary32 stores have kernels for groups of 8, 16, 32, 64, 128 and 256 elements only", group);
    return nullptr;
  }
  aq_handle* h = new (std::nothrow) aq_handle();
  if (!h) { fail(nullptr, AQ_ENOMEM, "host allocation failed"); return nullptr; }
  h->seq = seq; h->hidden = hidden; h->bits = bits; h->group = group;
  aq::State& st = h->st;
  st.n_samples = n_samples;
  st.elems = (long long)seq * hidden;
  st.chunks = (int)(st.elems / aq::kChunk);
  st.rows = (st.chunks + aq::kThreads - 1) / aq::kThreads;
  st.packed_bytes = st.elems * bits / 8;
  st.groups = st.elems / group;
  // any other multiple of 8 runs on the kernels of aq_anygroup.cu (lg_shift < 0 marks it)
  st.lanes_per_group = lanes ? lanes : group / aq::kChunk;
  st.lg_shift = lanes ? __builtin_ctz((unsigned)lanes) : -1;
  st.l2_prefetch = hosted ? 0 : h->l2_prefetch;     // rows in mapped host memory are not brought into L2
  cudaError_t e = cudaGetDevice(&h->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&st.sms, cudaDevAttrMultiProcessorCount, h->device);
  st.m_bits = m_bits;
  st.m_bytes = m_bits ? st.elems * m_bits / 8 : st.elems * 2;
  const size_t m_bytes = (size_t)n_samples * (size_t)st.m_bytes;
  const bool m_steps = m_bits == 2 || m_bits == 4 || m_bits == 8;
  const size_t m_scale_bytes = m_steps ? (size_t)n_samples * (size_t)st.groups * sizeof(float) : 0;
  const size_t seen_bytes = (size_t)n_samples * sizeof(unsigned long long);
  if (e == cudaSuccess && !hosted) e = cudaMalloc(&st.m, m_bytes);
  if (e == cudaSuccess && hosted) {
    // page-locked host memory that the GPU addresses directly: the kernels stream m over the bus
    e = cudaHostAlloc(&h->m_host, m_bytes, cudaHostAllocMapped | cudaHostAllocPortable);
    if (e == cudaSuccess) e = cudaHostGetDevicePointer(&st.m, h->m_host, 0);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&h->fetch_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&h->store_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_settled, cudaEventDisableTiming);
    for (aq_handle::Stage& sg : h->stage)
      for (cudaEvent_t* ev : {&sg.ev_staged, &sg.ev_computed, &sg.ev_written})
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming);
    for (int i = 0; i < aq_handle::kIdRing; ++i) {
      if (e == cudaSuccess) e = cudaHostAlloc(reinterpret_cast<void**>(&h->ids_pinned[i]), 2 * aq::kMaxBatch * sizeof(int32_t), cudaHostAllocPortable);
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_ids_sent[i], cudaEventDisableTiming);
    }
  }
  if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&st.seen), seen_bytes);
  if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&st.arrivals), sizeof(unsigned long long));
  if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&st.status), sizeof(uint32_t));
  if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&h->sum_dev), sizeof(unsigned long long));
  if (e == cudaSuccess && m_steps && !hosted) e = cudaMalloc(reinterpret_cast<void**>(&st.m_scales), m_scale_bytes);
  if (e == cudaSuccess && m_steps && hosted) {
    e = cudaHostAlloc(reinterpret_cast<void**>(&h->m_scales_host), m_scale_bytes, cudaHostAllocMapped | cudaHostAllocPortable);
    if (e == cudaSuccess) e = cudaHostGetDevicePointer(reinterpret_cast<void**>(&st.m_scales), h->m_scales_host, 0);
  }
  if (e == cudaSuccess && !hosted) e = cudaMemset(st.m, 0, m_bytes);           // Algorithm 1 starts from an all-zero m
  if (e == cudaSuccess && hosted) memset(h->m_host, 0, m_bytes);
  if (e == cudaSuccess && m_steps && !hosted) e = cudaMemset(st.m_scales, 0, m_scale_bytes);
  if (e == cudaSuccess && m_steps && hosted) memset(h->m_scales_host, 0, m_scale_bytes);
  if (e == cudaSuccess) e = cudaMemset(st.seen, 0, seen_bytes);
  if (e == cudaSuccess) e = cudaMemset(st.status, 0, sizeof(uint32_t));
  if (e == cudaSuccess) e = cudaMemset(st.arrivals, 0, sizeof(unsigned long long));
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    cuda_fail(nullptr, e, "aq_create");
    cudaGetLastError();
    aq_destroy(h);
    return nullptr;
  }
  return h;
}

void aq_destroy(aq_handle* h) {
  if (!h) return;
  DeviceGuard g(h->device);
  cudaStreamSynchronize(h->stream);
  free_staging(h);
  if (h->in_stream) {
    cudaStreamDestroy(h->in_stream); cudaStreamDestroy(h->out_stream);
    cudaEventDestroy(h->ev_begin);
    for (int i = 0; i < aq_handle::kSlices; ++i) { cudaEventDestroy(h->ev_in[i]); cudaEventDestroy(h->ev_done[i]); }
  }
  if (h->fetch_stream) {
    cudaStreamSynchronize(h->fetch_stream);
    cudaStreamSynchronize(h->store_stream);
    cudaStreamDestroy(h->fetch_stream);
    cudaStreamDestroy(h->store_stream);
    cudaEventDestroy(h->ev_settled);
    for (aq_handle::Stage& sg : h->stage) {
      cudaEventDestroy(sg.ev_staged); cudaEventDestroy(sg.ev_computed); cudaEventDestroy(sg.ev_written);
      cudaFree(sg.slots); cudaFree(sg.slot_scales); cudaFree(sg.d_slot_ids); cudaFree(sg.d_copy_ids);
    }
    for (int i = 0; i < aq_handle::kIdRing; ++i) {
      cudaFreeHost(h->ids_pinned[i]);
      cudaEventDestroy(h->ev_ids_sent[i]);
    }
  }
  if (h->m_host) cudaFreeHost(h->m_host);
  else cudaFree(h->st.m);
  if (h->m_scales_host) cudaFreeHost(h->m_scales_host);
  else cudaFree(h->st.m_scales);
  cudaFree(h->st.seen);
  cudaFree(h->st.arrivals);
  cudaFree(h->st.status);
  cudaFree(h->sum_dev);
  delete h;
}

int aq_configure(aq_handle* h, int key, int64_t value) {
  if (!h) return fail(nullptr, AQ_EINVAL, "null handle");
  switch (key) {
    case AQ_DTYPE:
      if (value != AQ_FP16 && value != AQ_BF16) return fail(h, AQ_EINVAL, "AQ_DTYPE must be AQ_FP16 or AQ_BF16");
      h->dtype = (int)value;
      return AQ_OK;
    case AQ_BATCH:
      if (value < 0 || value > aq::kMaxBatch) return fail(h, AQ_EINVAL, "AQ_BATCH must be in 0..%d", aq::kMaxBatch);
      h->n_batch = (int)value;
      return AQ_OK;
    case AQ_STREAM:
      h->stream = reinterpret_cast<cudaStream_t>(static_cast<intptr_t>(value));
      return AQ_OK;
    case AQ_RAW:
      if (value & 15) return fail(h, AQ_EINVAL, "AQ_RAW pointer must be 16-byte aligned");
      h->raw = reinterpret_cast<const void*>(static_cast<intptr_t>(value));
      return AQ_OK;
    case AQ_RAW_LIST:
      h->raw_list = reinterpret_cast<const void* const*>(static_cast<intptr_t>(value));
      return AQ_OK;
    case AQ_FIRST_FLAGS:
      h->first_flags = reinterpret_cast<uint8_t*>(static_cast<intptr_t>(value));
      return AQ_OK;
    case AQ_ROUNDING:
      if (value != AQ_ROUND_INTERVAL && value != AQ_ROUND_STOCHASTIC)
        return fail(h, AQ_EINVAL, "AQ_ROUNDING must be AQ_ROUND_INTERVAL or AQ_ROUND_STOCHASTIC");
      h->rounding = (int)value;
      return AQ_OK;
    case AQ_SEED:
      h->seed = (unsigned long long)value;
      return AQ_OK;
    case AQ_EPOCH:
      h->epoch = (unsigned long long)value;
      return AQ_OK;
    case AQ_L2_PREFETCH:
      if (value != 0 && value != 1) return fail(h, AQ_EINVAL, "AQ_L2_PREFETCH must be 0 or 1");
      h->l2_prefetch = (int)value;
      h->st.l2_prefetch = h->m_host ? 0 : (int)value;      // rows in mapped host memory are not brought into L2
      return AQ_OK;
    case AQ_ROWS_PER_CTA:
      if (value < 0 || value > (1 << 20)) return fail(h, AQ_EINVAL, "AQ_ROWS_PER_CTA must be in 0..2^20");
      h->st.rows_per_cta = (int)value;
      return AQ_OK;
    default:
      return fail(h, AQ_EINVAL, "unknown configure key %d", key);
  }
}

// The kernels of a call: the low-precision stores have their own, and so have the group sizes whose lanes
// are not a power of two within a warp.
static cudaError_t run_encode(aq_handle* h, const aq::State& st, const aq::EncodeArgs& a) {
  if (st.m_bits) return aq::launch_encode_lowbit(h->dtype, h->bits, st, a, h->stream);
  if (st.lg_shift < 0) return aq::launch_encode_anygroup(h->dtype, h->bits, st, a, h->stream);
  return aq::launch_encode(h->dtype, h->bits, st, a, h->stream);
}
static cudaError_t run_decode(aq_handle* h, const aq::State& st, const aq::DecodeArgs& a) {
  if (st.m_bits) return aq::launch_decode_lowbit(h->dtype, h->bits, st, a, h->stream);
  if (st.lg_shift < 0) return aq::launch_decode_anygroup(h->dtype, h->bits, st, a, h->stream);
  return aq::launch_decode(h->dtype, h->bits, st, a, h->stream);
}

static int launch_encode_call(aq_handle* h, const aq::EncodeArgs& a) {
  AQ_CUDA(h, settle(h));
  h->inplace_since_fetch = true;
  AQ_CUDA(h, run_encode(h, h->st, a));
  return AQ_OK;
}

static int launch_decode_call(aq_handle* h, const aq::DecodeArgs& a) {
  AQ_CUDA(h, settle(h));
  h->inplace_since_fetch = true;
  AQ_CUDA(h, run_decode(h, h->st, a));
  return AQ_OK;
}

static int encode_call(aq_handle* h, const void* act, const int32_t* sample_ids, void* packed, float* scales, bool lists,
                       const char* who) {
  if (!h) return fail(nullptr, AQ_EINVAL, "null handle");
  if (h->n_batch == 0) return AQ_OK;
  if (!act || !sample_ids || !packed || !scales) return fail(h, AQ_EINVAL, "%s: null pointer", who);
  if (!lists && (!aligned16(act) || !aligned16(packed) || !aligned16(scales)))
    return fail(h, AQ_EINVAL, "%s: act, packed and scales must be 16-byte aligned", who);
  if (lists && h->st.m_bits) return fail(h, AQ_EUNSUPPORTED, "%s: the list form is built for the 16-bit store only", who);
  DeviceGuard g(h->device);
  aq::EncodeArgs a{act, sample_ids, static_cast<uint8_t*>(packed), scales, h->first_flags, h->n_batch,
                   h->rounding == AQ_ROUND_STOCHASTIC, h->seed, h->epoch, lists};
  if (h->pending_stage >= 0)
    return run_staged(h, [&](const aq::State& st) { return run_encode(h, st, a); });
  return launch_encode_call(h, a);
}

int aq_encode(aq_handle* h, const void* act, const int32_t* sample_ids, void* packed, float* scales) {
  return encode_call(h, act, sample_ids, packed, scales, false, "aq_encode");
}

int aq_encode_list(aq_handle* h, const void* const* act_list, const int32_t* sample_ids, void* const* packed_list,
                   float* const* scales_list) {
  return encode_call(h, act_list, sample_ids, const_cast<void**>(packed_list),
                     reinterpret_cast<float*>(const_cast<float**>(scales_list)), true, "aq_encode_list");
}

static int decode_call(aq_handle* h, const void* packed, const float* scales, const int32_t* sample_ids, void* out, bool lists,
                       const char* who) {
  if (!h) return fail(nullptr, AQ_EINVAL, "null handle");
  if (h->n_batch == 0) return AQ_OK;
  if (!packed || !scales || !sample_ids || !out) return fail(h, AQ_EINVAL, "%s: null pointer", who);
  if (!lists && (!aligned16(packed) || !aligned16(scales) || !aligned16(out)))
    return fail(h, AQ_EINVAL, "%s: packed, scales and out must be 16-byte aligned", who);
  if (lists && h->st.m_bits) return fail(h, AQ_EUNSUPPORTED, "%s: the list form is built for the 16-bit store only", who);
  DeviceGuard g(h->device);
  aq::DecodeArgs a{static_cast<const uint8_t*>(packed), scales, lists ? static_cast<const void*>(h->raw_list) : h->raw, sample_ids,
                   out, h->first_flags, h->n_batch, lists};
  if (h->pending_stage >= 0)
    return run_staged(h, [&](const aq::State& st) { return run_decode(h, st, a); });
  return launch_decode_call(h, a);
}

int aq_decode(aq_handle* h, const void* packed, const float* scales, const int32_t* sample_ids, void* out) {
  return decode_call(h, packed, scales, sample_ids, out, false, "aq_decode");
}

int aq_decode_list(aq_handle* h, const void* const* packed_list, const float* const* scales_list, const int32_t* sample_ids,
                   void* const* out_list) {
  return decode_call(h, packed_list, reinterpret_cast<const float*>(scales_list), sample_ids, const_cast<void**>(out_list), true,
                     "aq_decode_list");
}

static int check_grad_args(aq_handle* h, const void* a, const void* b, const void* c, int64_t n_elems, int bits) {
  if (!h) return fail(nullptr, AQ_EINVAL, "null handle");
  if (bits < 1 || bits > 8) return fail(h, AQ_EINVAL, "bits must be in 1..8 (got %d)", bits);
  if (n_elems < 0 || n_elems % h->group) return fail(h, AQ_EINVAL, "n_elems must be a non-negative multiple of group %d", h->group);
  if (n_elems == 0) return AQ_OK;
  if (!a || !b || !c) return fail(h, AQ_EINVAL, "null pointer");
  if (!aligned16(a) || !aligned16(b) || !aligned16(c)) return fail(h, AQ_EINVAL, "pointers must be 16-byte aligned");
  return AQ_OK;
}

int aq_quant_grad(aq_handle* h, const void* grad, int64_t n_elems, int bits, void* packed, float* scales) {
  const int rc = check_grad_args(h, grad, packed, scales, n_elems, bits);
  if (rc != AQ_OK || n_elems == 0) return rc;
  DeviceGuard g(h->device);
  const bool stochastic = h->rounding == AQ_ROUND_STOCHASTIC;
  if (stochastic && n_elems / aq::kChunk > 0xFFFFFFFFll)
    return fail(h, AQ_EINVAL, "aq_quant_grad: stochastic rounding numbers chunks with 32 bits (n_elems < 2^35)");
  if (h->st.lg_shift < 0) {
    AQ_CUDA(h, aq::launch_quant_grad_anygroup(h->dtype, bits, h->st.lanes_per_group, grad, n_elems, static_cast<uint8_t*>(packed),
                                              scales, stochastic, h->seed, h->epoch, h->stream));
    return AQ_OK;
  }
  AQ_CUDA(h, aq::launch_quant_grad(h->dtype, bits, h->st.lanes_per_group, grad, n_elems,
                                   static_cast<uint8_t*>(packed), scales, stochastic, h->seed, h->epoch, h->l2_prefetch,
                                   h->stream));
  return AQ_OK;
}

int aq_dequant_grad(aq_handle* h, const void* packed, const float* scales, int64_t n_elems, int bits, void* out) {
  const int rc = check_grad_args(h, packed, scales, out, n_elems, bits);
  if (rc != AQ_OK || n_elems == 0) return rc;
  DeviceGuard g(h->device);
  if (h->st.lg_shift < 0) {
    AQ_CUDA(h, aq::launch_dequant_grad_anygroup(h->dtype, bits, h->st.lanes_per_group, static_cast<const uint8_t*>(packed), scales,
                                                n_elems, out, h->stream));
    return AQ_OK;
  }
  AQ_CUDA(h, aq::launch_dequant_grad(h->dtype, bits, h->st.lanes_per_group, static_cast<const uint8_t*>(packed),
                                     scales, n_elems, out, h->stream));
  return AQ_OK;
}

int aq_state_checksum(aq_handle* h, uint64_t* out_host) {
  if (!h) return fail(nullptr, AQ_EINVAL, "null handle");
  if (!out_host) return fail(h, AQ_EINVAL, "aq_state_checksum: null pointer");
  DeviceGuard g(h->device);
  AQ_CUDA(h, settle(h));
  AQ_CUDA(h, cudaMemsetAsync(h->sum_dev, 0, sizeof(unsigned long long), h->stream));
  AQ_CUDA(h, aq::launch_checksum(h->st, h->sum_dev, h->stream));
  unsigned long long v = 0;
  AQ_CUDA(h, cudaMemcpyAsync(&v, h->sum_dev, sizeof(v), cudaMemcpyDeviceToHost, h->stream));
  AQ_CUDA(h, cudaStreamSynchronize(h->stream));
  *out_host = v;
  return AQ_OK;
}

int aq_status(aq_handle* h, uint32_t* bits_host) {
  if (!h) return fail(nullptr, AQ_EINVAL, "null handle");
  if (!bits_host) return fail(h, AQ_EINVAL, "aq_status: null pointer");
  DeviceGuard g(h->device);
  uint32_t v = 0;
  AQ_CUDA(h, cudaMemcpyAsync(&v, h->st.status, sizeof(v), cudaMemcpyDeviceToHost, h->stream));
  AQ_CUDA(h, cudaMemsetAsync(h->st.status, 0, sizeof(uint32_t), h->stream));
  AQ_CUDA(h, cudaStreamSynchronize(h->stream));
  *bits_host = v;
  return AQ_OK;
}

const char* aq_last_error(aq_handle* h) { return h ? h->err : g_create_err; }
int aq_last_error_code(aq_handle* h) { return h ? h->err_code : g_create_code; }

int64_t aq_packed_bytes_per_sample(aq_handle* h) { return h ? h->st.packed_bytes : 0; }
int64_t aq_scales_per_sample(aq_handle* h) { return h ? h->st.groups : 0; }
int64_t aq_m_bytes_per_sample(aq_handle* h) {
  if (!h) return 0;
  return h->st.m_bytes + (h->st.m_scales ? h->st.groups * (int64_t)sizeof(float) : 0);
}

// slice i of kSlices over n samples: [lo, lo + cnt)
static void slice_of(int n, int i, size_t* lo, size_t* cnt) {
  const int base = n / aq_handle::kSlices, rest = n % aq_handle::kSlices;
  *lo = (size_t)i * base + (size_t)(i < rest ? i : rest);
  *cnt = (size_t)base + (i < rest ? 1 : 0);
}

int aq_encode_host(aq_handle* h, const void* act_host, const int32_t* sample_ids_host, void* packed_host,
                   float* scales_host) {
  if (!h) return fail(nullptr, AQ_EINVAL, "null handle");
  if (h->n_batch == 0) return AQ_OK;
  if (!act_host || !sample_ids_host || !packed_host || !scales_host) return fail(h, AQ_EINVAL, "aq_encode_host: null pointer");
  DeviceGuard g(h->device);
  int rc = ensure_staging(h);
  if (rc != AQ_OK) return rc;
  const size_t nb = (size_t)h->n_batch;
  const size_t act_b = (size_t)h->st.elems * 2, packed_b = (size_t)h->st.packed_bytes, scales_b = (size_t)h->st.groups * sizeof(float);
  if (!sliceable(h, sample_ids_host)) {
    AQ_CUDA(h, cudaMemcpyAsync(h->d_act, act_host, nb * act_b, cudaMemcpyHostToDevice, h->stream));
    AQ_CUDA(h, cudaMemcpyAsync(h->d_ids, sample_ids_host, nb * sizeof(int32_t), cudaMemcpyHostToDevice, h->stream));
    rc = aq_encode(h, h->d_act, h->d_ids, h->d_packed, h->d_scales);
    if (rc != AQ_OK) return rc;
    AQ_CUDA(h, cudaMemcpyAsync(packed_host, h->d_packed, nb * packed_b, cudaMemcpyDeviceToHost, h->stream));
    AQ_CUDA(h, cudaMemcpyAsync(scales_host, h->d_scales, nb * scales_b, cudaMemcpyDeviceToHost, h->stream));
    AQ_CUDA(h, cudaStreamSynchronize(h->stream));
    return AQ_OK;
  }
  rc = ensure_slicing(h);
  if (rc != AQ_OK) return rc;
  AQ_CUDA(h, cudaEventRecord(h->ev_begin, h->stream));          // the staging block is free once earlier work is done
  AQ_CUDA(h, cudaStreamWaitEvent(h->in_stream, h->ev_begin, 0));
  AQ_CUDA(h, cudaMemcpyAsync(h->d_ids, sample_ids_host, nb * sizeof(int32_t), cudaMemcpyHostToDevice, h->in_stream));
  for (int i = 0; i < aq_handle::kSlices; ++i) {
    size_t lo, cnt;
    slice_of(h->n_batch, i, &lo, &cnt);
    char* d_act = static_cast<char*>(h->d_act) + lo * act_b;
    AQ_CUDA(h, cudaMemcpyAsync(d_act, static_cast<const char*>(act_host) + lo * act_b, cnt * act_b, cudaMemcpyHostToDevice, h->in_stream));
    AQ_CUDA(h, cudaEventRecord(h->ev_in[i], h->in_stream));
    AQ_CUDA(h, cudaStreamWaitEvent(h->stream, h->ev_in[i], 0));
    const aq::EncodeArgs a{d_act, h->d_ids + lo, h->d_packed + lo * packed_b, h->d_scales + lo * (size_t)h->st.groups,
                           h->first_flags ? h->first_flags + lo : nullptr, (int)cnt,
                           h->rounding == AQ_ROUND_STOCHASTIC, h->seed, h->epoch};
    rc = launch_encode_call(h, a);
    if (rc != AQ_OK) return rc;
    AQ_CUDA(h, cudaEventRecord(h->ev_done[i], h->stream));
    AQ_CUDA(h, cudaStreamWaitEvent(h->out_stream, h->ev_done[i], 0));
    AQ_CUDA(h, cudaMemcpyAsync(static_cast<char*>(packed_host) + lo * packed_b, h->d_packed + lo * packed_b, cnt * packed_b,
                               cudaMemcpyDeviceToHost, h->out_stream));
    AQ_CUDA(h, cudaMemcpyAsync(reinterpret_cast<char*>(scales_host) + lo * scales_b, h->d_scales + lo * (size_t)h->st.groups,
                               cnt * scales_b, cudaMemcpyDeviceToHost, h->out_stream));
  }
  AQ_CUDA(h, cudaStreamSynchronize(h->out_stream));
  return AQ_OK;
}

int aq_decode_host(aq_handle* h, const void* packed_host, const float* scales_host, const void* raw_host,
                   const int32_t* sample_ids_host, void* out_host) {
  if (!h) return fail(nullptr, AQ_EINVAL, "null handle");
  if (h->n_batch == 0) return AQ_OK;
  if (!packed_host || !scales_host || !sample_ids_host || !out_host) return fail(h, AQ_EINVAL, "aq_decode_host: null pointer");
  DeviceGuard g(h->device);
  int rc = ensure_staging(h);
  if (rc != AQ_OK) return rc;
  const size_t nb = (size_t)h->n_batch;
  const size_t act_b = (size_t)h->st.elems * 2, packed_b = (size_t)h->st.packed_bytes, scales_b = (size_t)h->st.groups * sizeof(float);
  // the staging block holds the raw message on the way in and the activation on the way out
  // (every element is read before the same thread overwrites it)
  if (!sliceable(h, sample_ids_host)) {
    AQ_CUDA(h, cudaMemcpyAsync(h->d_packed, packed_host, nb * packed_b, cudaMemcpyHostToDevice, h->stream));
    AQ_CUDA(h, cudaMemcpyAsync(h->d_scales, scales_host, nb * scales_b, cudaMemcpyHostToDevice, h->stream));
    AQ_CUDA(h, cudaMemcpyAsync(h->d_ids, sample_ids_host, nb * sizeof(int32_t), cudaMemcpyHostToDevice, h->stream));
    if (raw_host) AQ_CUDA(h, cudaMemcpyAsync(h->d_act, raw_host, nb * act_b, cudaMemcpyHostToDevice, h->stream));
    const void* saved_raw = h->raw;
    h->raw = raw_host ? h->d_act : nullptr;
    rc = aq_decode(h, h->d_packed, h->d_scales, h->d_ids, h->d_act);
    h->raw = saved_raw;
    if (rc != AQ_OK) return rc;
    AQ_CUDA(h, cudaMemcpyAsync(out_host, h->d_act, nb * act_b, cudaMemcpyDeviceToHost, h->stream));
    AQ_CUDA(h, cudaStreamSynchronize(h->stream));
    return AQ_OK;
  }
  rc = ensure_slicing(h);
  if (rc != AQ_OK) return rc;
  AQ_CUDA(h, cudaEventRecord(h->ev_begin, h->stream));
  AQ_CUDA(h, cudaStreamWaitEvent(h->in_stream, h->ev_begin, 0));
  AQ_CUDA(h, cudaMemcpyAsync(h->d_ids, sample_ids_host, nb * sizeof(int32_t), cudaMemcpyHostToDevice, h->in_stream));
  for (int i = 0; i < aq_handle::kSlices; ++i) {
    size_t lo, cnt;
    slice_of(h->n_batch, i, &lo, &cnt);
    char* d_act = static_cast<char*>(h->d_act) + lo * act_b;
    AQ_CUDA(h, cudaMemcpyAsync(h->d_packed + lo * packed_b, static_cast<const char*>(packed_host) + lo * packed_b, cnt * packed_b,
                               cudaMemcpyHostToDevice, h->in_stream));
    AQ_CUDA(h, cudaMemcpyAsync(h->d_scales + lo * (size_t)h->st.groups, reinterpret_cast<const char*>(scales_host) + lo * scales_b,
                               cnt * scales_b, cudaMemcpyHostToDevice, h->in_stream));
    if (raw_host)
      AQ_CUDA(h, cudaMemcpyAsync(d_act, static_cast<const char*>(raw_host) + lo * act_b, cnt * act_b, cudaMemcpyHostToDevice, h->in_stream));
    AQ_CUDA(h, cudaEventRecord(h->ev_in[i], h->in_stream));
    AQ_CUDA(h, cudaStreamWaitEvent(h->stream, h->ev_in[i], 0));
    const aq::DecodeArgs a{h->d_packed + lo * packed_b, h->d_scales + lo * (size_t)h->st.groups, raw_host ? d_act : nullptr,
                           h->d_ids + lo, d_act, h->first_flags ? h->first_flags + lo : nullptr, (int)cnt};
    rc = launch_decode_call(h, a);
    if (rc != AQ_OK) return rc;
    AQ_CUDA(h, cudaEventRecord(h->ev_done[i], h->stream));
    AQ_CUDA(h, cudaStreamWaitEvent(h->out_stream, h->ev_done[i], 0));
    AQ_CUDA(h, cudaMemcpyAsync(static_cast<char*>(out_host) + lo * act_b, d_act, cnt * act_b, cudaMemcpyDeviceToHost, h->out_stream));
  }
  AQ_CUDA(h, cudaStreamSynchronize(h->out_stream));
  return AQ_OK;
}

int aq_prefetch(aq_handle* h, const int32_t* sample_ids_host, int n) {
  if (!h) return fail(nullptr, AQ_EINVAL, "null handle");
  if (!h->m_host) return fail(h, AQ_EUNSUPPORTED, "aq_prefetch: the handle keeps m in device memory (see aq_create_hosted)");
  if (n != h->n_batch) return fail(h, AQ_EINVAL, "aq_prefetch: n must equal AQ_BATCH (%d), got %d", h->n_batch, n);
  if (n == 0) return AQ_OK;
  if (!sample_ids_host) return fail(h, AQ_EINVAL, "aq_prefetch: null pointer");
  DeviceGuard g(h->device);
  const size_t bytes = (size_t)h->st.m_bytes;
  // a prefetch that replaces a pending one reuses its block; otherwise the blocks take turns
  const int which = h->pending_stage >= 0 ? h->pending_stage : h->next_stage;
  aq_handle::Stage& sg = h->stage[which];
  aq_handle::Stage& other = h->stage[1 - which];
  if (sg.batch < n) {
    AQ_CUDA(h, cudaStreamSynchronize(h->fetch_stream));
    AQ_CUDA(h, cudaStreamSynchronize(h->store_stream));
    AQ_CUDA(h, cudaStreamSynchronize(h->stream));
    cudaFree(sg.slots); cudaFree(sg.slot_scales); cudaFree(sg.d_slot_ids); cudaFree(sg.d_copy_ids);
    sg.slots = nullptr; sg.slot_scales = nullptr; sg.d_slot_ids = nullptr; sg.d_copy_ids = nullptr; sg.batch = 0;
    AQ_CUDA(h, cudaMalloc(&sg.slots, (size_t)n * bytes));
    if (h->m_scales_host)
      AQ_CUDA(h, cudaMalloc(reinterpret_cast<void**>(&sg.slot_scales), (size_t)n * (size_t)h->st.groups * sizeof(float)));
    AQ_CUDA(h, cudaMalloc(reinterpret_cast<void**>(&sg.d_slot_ids), (size_t)n * sizeof(int32_t)));
    AQ_CUDA(h, cudaMalloc(reinterpret_cast<void**>(&sg.d_copy_ids), (size_t)n * sizeof(int32_t)));
    sg.batch = n;
  }
  // rows to move: every id once (the kernels skip an id's later occurrences and ids out of range)
  sg.ids.assign(sample_ids_host, sample_ids_host + n);
  std::unordered_set<int32_t> taken;
  for (int32_t& id : sg.ids)
    if (id < 0 || (long long)id >= h->st.n_samples || !taken.insert(id).second) id = -1;
  // What the copies have to wait for, on the device: the block's own rows of two calls ago going home;
  // the other block's rows going home when that call updates a sample that is fetched again here;
  // and, when a call has worked on the host block in place since the last prefetch, everything
  // issued so far on the handle's stream.  Not the call that is computing on the other block.
  if (sg.writeback_issued) AQ_CUDA(h, cudaStreamWaitEvent(h->fetch_stream, sg.ev_written, 0));
  if (other.writeback_issued) {
    bool shared = false;
    for (int32_t id : other.ids) shared = shared || (id >= 0 && taken.count(id));
    if (shared) AQ_CUDA(h, cudaStreamWaitEvent(h->fetch_stream, other.ev_written, 0));
  }
  if (h->inplace_since_fetch) {
    AQ_CUDA(h, cudaEventRecord(h->ev_settled, h->stream));
    AQ_CUDA(h, cudaStreamWaitEvent(h->fetch_stream, h->ev_settled, 0));
    h->inplace_since_fetch = false;
  }
  const int ring = (int)(h->prefetches++ % aq_handle::kIdRing);
  AQ_CUDA(h, cudaEventSynchronize(h->ev_ids_sent[ring]));      // long done, unless kIdRing prefetches are queued
  int32_t* copy_ids_pinned = h->ids_pinned[ring] + aq::kMaxBatch;
  memcpy(h->ids_pinned[ring], sample_ids_host, (size_t)n * sizeof(int32_t));
  memcpy(copy_ids_pinned, sg.ids.data(), (size_t)n * sizeof(int32_t));
  AQ_CUDA(h, cudaMemcpyAsync(sg.d_slot_ids, h->ids_pinned[ring], (size_t)n * sizeof(int32_t), cudaMemcpyHostToDevice, h->fetch_stream));
  AQ_CUDA(h, cudaMemcpyAsync(sg.d_copy_ids, copy_ids_pinned, (size_t)n * sizeof(int32_t), cudaMemcpyHostToDevice, h->fetch_stream));
  AQ_CUDA(h, cudaEventRecord(h->ev_ids_sent[ring], h->fetch_stream));
  // a few large rows: one copy per row through the copy engines, the faster way over the host
  // link; many rows or small ones: one kernel that reads the mapped host block, since a copy
  // call costs microseconds of host time each
  sg.rows_by_kernel = n > 64 || bytes < (64u << 10);
  const int rc = move_rows(h, sg, true, h->fetch_stream);
  if (rc != AQ_OK) return rc;
  AQ_CUDA(h, cudaEventRecord(sg.ev_staged, h->fetch_stream));
  if (h->pending_stage < 0) h->next_stage = 1 - which;
  h->pending_stage = which;
  return AQ_OK;
}

// The byte ranges of a message from the handle's device to dst_device, on the handle's stream: one
// kernel launch when both ends are on the handle's device and every range is made of whole,
// aligned 16-byte pieces; otherwise one copy per range (peer copies into the receiver's memory).
static int wire_ranges(aq_handle* h, int dst_device, const void* const* src, void* const* dst, const size_t* bytes, int n) {
  bool by_kernel = dst_device == h->device;
  for (int k = 0; k < n; ++k)
    by_kernel = by_kernel && bytes[k] % 16 == 0 && aligned16(src[k]) && aligned16(dst[k]);
  if (by_kernel) {
    AQ_CUDA(h, aq::launch_wire_copy(src, dst, bytes, n, h->stream));
    return AQ_OK;
  }
  for (int k = 0; k < n; ++k)
    AQ_CUDA(h, cudaMemcpyPeerAsync(dst[k], dst_device, src[k], h->device, bytes[k], h->stream));
  return AQ_OK;
}

int aq_wire_copy(aq_handle* h, int dst_device, void* packed_dst, float* scales_dst, void* raw_dst,
                 const void* packed_src, const float* scales_src, const void* raw_src) {
  if (!h) return fail(nullptr, AQ_EINVAL, "null handle");
  if (h->n_batch == 0) return AQ_OK;
  if (!packed_dst || !scales_dst || !packed_src || !scales_src) return fail(h, AQ_EINVAL, "aq_wire_copy: null pointer");
  if ((raw_dst == nullptr) != (raw_src == nullptr)) return fail(h, AQ_EINVAL, "aq_wire_copy: raw_dst and raw_src go together");
  int n_dev = 0;
  AQ_CUDA(h, cudaGetDeviceCount(&n_dev));
  if (dst_device < 0 || dst_device >= n_dev) return fail(h, AQ_EINVAL, "aq_wire_copy: no device %d", dst_device);
  DeviceGuard g(h->device);
  const size_t nb = (size_t)h->n_batch;
  const void* src[3] = {packed_src, scales_src, raw_src};
  void* dst[3] = {packed_dst, scales_dst, raw_dst};
  const size_t bytes[3] = {nb * (size_t)h->st.packed_bytes, nb * (size_t)h->st.groups * sizeof(float), nb * (size_t)h->st.elems * 2};
  return wire_ranges(h, dst_device, src, dst, bytes, raw_src ? 3 : 2);
}

int aq_wire_copy_grad(aq_handle* h, int dst_device, void* packed_dst, float* scales_dst, const void* packed_src,
                      const float* scales_src, int64_t n_elems, int bits) {
  if (!h) return fail(nullptr, AQ_EINVAL, "null handle");
  if (bits < 1 || bits > 8) return fail(h, AQ_EINVAL, "bits must be in 1..8 (got %d)", bits);
  if (n_elems < 0 || n_elems % h->group) return fail(h, AQ_EINVAL, "n_elems must be a non-negative multiple of group %d", h->group);
  if (n_elems == 0) return AQ_OK;
  if (!packed_dst || !scales_dst || !packed_src || !scales_src) return fail(h, AQ_EINVAL, "aq_wire_copy_grad: null pointer");
  int n_dev = 0;
  AQ_CUDA(h, cudaGetDeviceCount(&n_dev));
  if (dst_device < 0 || dst_device >= n_dev) return fail(h, AQ_EINVAL, "aq_wire_copy_grad: no device %d", dst_device);
  DeviceGuard g(h->device);
  const void* src[2] = {packed_src, scales_src};
  void* dst[2] = {packed_dst, scales_dst};
  const size_t bytes[2] = {(size_t)n_elems * (size_t)bits / 8, (size_t)(n_elems / h->group) * sizeof(float)};
  return wire_ranges(h, dst_device, src, dst, bytes, 2);
}

int aq_export_sample(aq_handle* h, int64_t sample_id, void* m_host, uint8_t* seen_host) {
  if (!h) return fail(nullptr, AQ_EINVAL, "null handle");
  if (sample_id < 0 || sample_id >= h->st.n_samples) return fail(h, AQ_EINVAL, "sample id out of range");
  if (!m_host && !seen_host) return fail(h, AQ_EINVAL, "aq_export_sample: null pointers");
  DeviceGuard g(h->device);
  AQ_CUDA(h, settle(h));
  const size_t bytes = (size_t)h->st.m_bytes;
  if (m_host) {
    AQ_CUDA(h, cudaMemcpyAsync(m_host, static_cast<const char*>(h->st.m) + (size_t)sample_id * bytes, bytes,
                               cudaMemcpyDeviceToHost, h->stream));
    if (h->st.m_scales)                           // the steps follow the codes
      AQ_CUDA(h, cudaMemcpyAsync(static_cast<char*>(m_host) + bytes, h->st.m_scales + (size_t)sample_id * h->st.groups,
                                 (size_t)h->st.groups * sizeof(float), cudaMemcpyDeviceToHost, h->stream));
  }
  unsigned long long stamp = 0;
  if (seen_host)
    AQ_CUDA(h, cudaMemcpyAsync(&stamp, h->st.seen + sample_id, sizeof(stamp), cudaMemcpyDeviceToHost, h->stream));
  AQ_CUDA(h, cudaStreamSynchronize(h->stream));
  if (seen_host) *seen_host = stamp != 0 ? 1 : 0;
  return AQ_OK;
}

int aq_import_sample(aq_handle* h, int64_t sample_id, const void* m_host, uint8_t seen) {
  if (!h) return fail(nullptr, AQ_EINVAL, "null handle");
  if (sample_id < 0 || sample_id >= h->st.n_samples) return fail(h, AQ_EINVAL, "sample id out of range");
  if (!m_host) return fail(h, AQ_EINVAL, "aq_import_sample: null pointer");
  DeviceGuard g(h->device);
  AQ_CUDA(h, settle(h));
  h->inplace_since_fetch = true;
  const size_t bytes = (size_t)h->st.m_bytes;
  const unsigned long long stamp = seen ? aq::kImportedStamp : 0ull;
  AQ_CUDA(h, cudaMemcpyAsync(static_cast<char*>(h->st.m) + (size_t)sample_id * bytes, m_host, bytes,
                             cudaMemcpyHostToDevice, h->stream));
  if (h->st.m_scales)
    AQ_CUDA(h, cudaMemcpyAsync(h->st.m_scales + (size_t)sample_id * h->st.groups, static_cast<const char*>(m_host) + bytes,
                               (size_t)h->st.groups * sizeof(float), cudaMemcpyHostToDevice, h->stream));
  AQ_CUDA(h, cudaMemcpyAsync(h->st.seen + sample_id, &stamp, sizeof(stamp), cudaMemcpyHostToDevice, h->stream));
  AQ_CUDA(h, cudaStreamSynchronize(h->stream));
  return AQ_OK;
}

}  // extern "C"

// ---- access for entry points that live in other files of the library

namespace aq {

const State* handle_state(aq_handle* h) { return &h->st; }
cudaStream_t handle_stream(aq_handle* h) { return h->stream; }
int handle_device(aq_handle* h) { return h->device; }

int handle_fail(aq_handle* h, int code, const char* msg) { return fail(h, code, "%s", msg); }
cudaError_t handle_settle(aq_handle* h) { return settle(h); }

}  // namespace aq

