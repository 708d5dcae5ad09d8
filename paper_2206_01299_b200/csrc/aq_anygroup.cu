// Kernels for group sizes that the main kernels do not take: any multiple of 8 elements whose
// lane count (group / 8) is not a power of two up to 32 -- groups of 24, 40, 48, 96 ... elements, and
// groups longer than 256 up to a whole hidden row.  The quantizer (Section 4.1 "Baselines", per
// group: largest magnitude, 2^b intervals) is the one of aq_device.cuh; what differs is which lanes
// share a group.
//
// Sender side and gradient quantizer: the L = group / 8 chunks of a group go to a tile of
// W = min(32, next power of two >= L) lanes of one warp, lane t of the tile taking chunks t, t + W,
// ... of its group; a warp holds 32 / W groups at a time and the group maximum is a shuffle
// butterfly over the tile (idle lanes contribute 0).  A lane that has more than one chunk
// (groups of more than 256 elements) reads its later chunks a second time after the maximum is
// known.  Receiver side and gradient dequantizer need no reduction: one chunk per lane as in the
// main kernels, with the group of a chunk found by a division.  Codes go through the byte-wise
// path of store_codes / load_codes.  None of this is tuned: these shapes are outside the measured
// workloads; the results are bit for bit those of the definition, like everywhere else.

#include "aq_device.cuh"

namespace aq {
namespace {

struct Tiling {
  int lanes;            // L: chunks per group
  int width;            // W: lanes of a tile
  int per_lane;         // ceil(L / W): chunks a lane takes from its group
  int groups_per_warp;  // 32 / W
};

inline Tiling tiling_for(int lanes_per_group) {
  Tiling t;
  t.lanes = lanes_per_group;
  t.width = 1;
  while (t.width < lanes_per_group && t.width < 32) t.width *= 2;
  t.per_lane = (lanes_per_group + t.width - 1) / t.width;
  t.groups_per_warp = 32 / t.width;
  return t;
}

constexpr int kWarps = kThreads / 32;

__device__ __forceinline__ float tile_max(float s, int width) {
  for (int o = width >> 1; o > 0; o >>= 1) s = fmaxf(s, __shfl_xor_sync(kFullMask, s, o));
  return s;
}

// Groups [g_lo, g_hi) of one stream of groups (a sample, or a call's gradient), numbered from the
// base pointers: quantizes `in` (minus m, when m is given) and writes codes, steps and the new m.
// Every lane of the CTA runs the same number of iterations (the shuffles and votes inside need
// all of them); lanes without a chunk work on zeros and store nothing.
template <typename T, int BITS, bool STOCH, bool WITH_M>
__device__ __forceinline__ void quantize_groups(const Tiling tl, const T* __restrict__ in, T* __restrict__ m,
                                                uint8_t* __restrict__ stream, float* __restrict__ scales,
                                                long long g_lo, long long g_hi, unsigned long long seed,
                                                unsigned long long epoch, uint32_t stream_id) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int tile = lane / tl.width, t = lane - tile * tl.width;
  for (long long gb = g_lo + (long long)warp * tl.groups_per_warp; gb < g_hi; gb += (long long)kWarps * tl.groups_per_warp) {
    const long long g = gb + tile;
    const bool have_group = g < g_hi;
    const long long c_first = g * tl.lanes + t;
    // pass 1: the group's largest magnitude; the lane's first chunk stays in registers
    uint4 a0 = make_uint4(0, 0, 0, 0), m0 = make_uint4(0, 0, 0, 0);
    float s = 0.0f;
    for (int k = 0; k < tl.per_lane; ++k) {
      const int ck = t + k * tl.width;
      const bool active = have_group && ck < tl.lanes;
      const long long c = c_first + (long long)k * tl.width;
      uint4 av = make_uint4(0, 0, 0, 0), mv = make_uint4(0, 0, 0, 0);
      if (active) {
        av = ld_stream(in + c * kChunk);
        if (WITH_M) mv = ld_stream(m + c * kChunk);
      }
      if (k == 0) {
        a0 = av;
        m0 = mv;
      }
      float mf[8], d[8];
      Conv<T>::unpack(mv, mf);
      Conv<T>::diff(av, mf, d);
      s = fmaxf(s, abs_max8(d));
    }
    s = tile_max(s, tl.width);
    // pass 2: codes, step, new m
    for (int k = 0; k < tl.per_lane; ++k) {
      const int ck = t + k * tl.width;
      const bool active = have_group && ck < tl.lanes;
      const long long c = c_first + (long long)k * tl.width;
      uint4 av = a0, mv = m0;
      if (k > 0) {
        av = mv = make_uint4(0, 0, 0, 0);
        if (active) {
          av = __ldcg(reinterpret_cast<const uint4*>(in + c * kChunk));
          if (WITH_M) mv = __ldcg(reinterpret_cast<const uint4*>(m + c * kChunk));
        }
      }
      float mf[8], d[8], q[8];
      Conv<T>::unpack(mv, mf);
      Conv<T>::diff(av, mf, d);
      float delta;
      unsigned long long codes;
      uint4 noise = make_uint4(0, 0, 0, 0);
      if constexpr (STOCH) noise = chunk_noise(seed, epoch, stream_id, (uint32_t)c);
      quantize8_for<BITS, Conv<T>::kWide, STOCH>(d, s, noise, delta, codes, q);
      if (active) {
        if (WITH_M) {
#pragma unroll
          for (int j = 0; j < 8; ++j) mf[j] = __fadd_rn(mf[j], q[j]);
          st_stream(m + c * kChunk, Conv<T>::pack(mf));
        }
        if (ck == 0) scales[g] = delta;
      }
      store_codes<BITS>(stream, c, lane, active, false, codes);
    }
  }
}

// groups of a sample (or of a gradient) that one CTA takes: about four rows' worth of chunks, a
// whole number of warp loads
inline long long groups_per_cta(const Tiling& tl) {
  const long long per_pass = (long long)kWarps * tl.groups_per_warp;
  long long passes = (4 * kThreads) / (per_pass * tl.lanes);
  if (passes < 1) passes = 1;
  return per_pass * passes;
}

template <typename T, int BITS, bool STOCH>
__global__ void __launch_bounds__(kThreads) encode_anygroup_kernel(const State st, const EncodeArgs a, const LaunchPlan plan,
                                                                   const Tiling tl, const long long per_cta) {
  const int y = blockIdx.y;
  overlap_with_neighbours();
  const BufferLists lists = {{a.act_list(), a.packed_list(), a.scales_list(), nullptr}, {true, true, true, false}};
  const Sample sample = open_sample(st, plan, a.ids, y, false, false, a.first_flags, a.lists ? &lists : nullptr);
  const unsigned long long elems = (unsigned long long)st.elems;
  // the sample's buffers: at a fixed stride from the call's base pointers, or (list form) fetched with the sample
  const T* act = reinterpret_cast<const T*>(a.act) + (unsigned long long)(unsigned)y * elems;
  uint8_t* stream = a.packed + (unsigned long long)(unsigned)y * (unsigned long long)st.packed_bytes;
  float* scales = a.scales + (unsigned long long)(unsigned)y * (unsigned long long)st.groups;
  if (a.lists) {
    if (sample.mode == kModeNothing) return;
    act = static_cast<const T*>(sample.buf[0]);
    stream = static_cast<uint8_t*>(const_cast<void*>(sample.buf[1]));
    scales = static_cast<float*>(const_cast<void*>(sample.buf[2]));
  }
  const long long g_lo = (long long)blockIdx.x * per_cta;
  const long long g_hi = g_lo + per_cta < st.groups ? g_lo + per_cta : st.groups;
  if (sample.mode == kModeDelta) {
    T* m = reinterpret_cast<T*>(st.m) + (unsigned long long)sample.row * elems;
    quantize_groups<T, BITS, STOCH, true>(tl, act, m, stream, scales, g_lo, g_hi, a.seed, a.epoch, (uint32_t)sample.id);
  } else {
    // first visit: the activation itself becomes m(xi); skipped sample: nothing is stored.  Either
    // way the sample's codes and steps are zero.
    T* m = (sample.mode == kModeFirst) ? reinterpret_cast<T*>(st.m) + (unsigned long long)sample.row * elems : nullptr;
    const int lane = threadIdx.x & 31;
    for (long long c = g_lo * tl.lanes + threadIdx.x; c < g_hi * tl.lanes; c += kThreads) {
      if (m) st_stream(m + c * kChunk, ld_stream(act + c * kChunk));
      store_codes<BITS>(stream, c, lane, true, false, 0ull);
    }
    for (long long g = g_lo + threadIdx.x; g < g_hi; g += kThreads) scales[g] = 0.0f;
  }
}

template <typename T, int BITS>
__global__ void __launch_bounds__(kThreads) decode_anygroup_kernel(const State st, const DecodeArgs a, const LaunchPlan plan,
                                                                   const int lanes_per_group, const long long per_cta) {
  const int y = blockIdx.y;
  const int lane = threadIdx.x & 31;
  overlap_with_neighbours();
  const BufferLists lists = {{a.packed_list(), a.scales_list(), a.raw_list(), a.out_list()}, {true, true, false, true}};
  const Sample sample = open_sample(st, plan, a.ids, y, true, a.raw != nullptr, a.first_flags, a.lists ? &lists : nullptr,
                                    a.raw != nullptr ? 2 : -1);
  const unsigned long long elems = (unsigned long long)st.elems;
  T* out = reinterpret_cast<T*>(a.out) + (unsigned long long)(unsigned)y * elems;
  const uint8_t* stream = a.packed + (unsigned long long)(unsigned)y * (unsigned long long)st.packed_bytes;
  const float* scales = a.scales + (unsigned long long)(unsigned)y * (unsigned long long)st.groups;
  const T* raw = a.raw ? reinterpret_cast<const T*>(a.raw) + (unsigned long long)(unsigned)y * elems : nullptr;
  if (a.lists) {
    if (sample.mode == kModeNothing) return;
    stream = static_cast<const uint8_t*>(sample.buf[0]);
    scales = static_cast<const float*>(sample.buf[1]);
    raw = static_cast<const T*>(sample.buf[2]);
    out = static_cast<T*>(const_cast<void*>(sample.buf[3]));
  }
  const long long g_lo = (long long)blockIdx.x * per_cta;
  const long long g_hi = g_lo + per_cta < st.groups ? g_lo + per_cta : st.groups;
  const long long c_lo = g_lo * lanes_per_group, c_hi = g_hi * lanes_per_group;
  if (sample.mode == kModeDelta) {
    T* m = reinterpret_cast<T*>(st.m) + (unsigned long long)sample.row * elems;
    for (long long c = c_lo + threadIdx.x; c < c_hi; c += kThreads) {
      const uint4 mv = ld_stream(m + c * kChunk);
      const float delta = __ldg(scales + c / lanes_per_group);
      const unsigned long long codes = load_codes<BITS>(stream, c, lane, true, false);
      float mf[8], q[8];
      Conv<T>::unpack(mv, mf);
      dequantize8<BITS>(codes, delta, q);
#pragma unroll
      for (int j = 0; j < 8; ++j) mf[j] = __fadd_rn(mf[j], q[j]);
      const uint4 nv = Conv<T>::pack(mf);
      st_stream(m + c * kChunk, nv);
      st_stream(out + c * kChunk, nv);
    }
  } else {
    // first visit: the raw message becomes m(xi) and the activation; skipped sample: zeros out
    const bool first = sample.mode == kModeFirst;
    T* m = first ? reinterpret_cast<T*>(st.m) + (unsigned long long)sample.row * elems : nullptr;
    for (long long c = c_lo + threadIdx.x; c < c_hi; c += kThreads) {
      uint4 v = make_uint4(0, 0, 0, 0);
      if (first) {
        v = ld_stream(raw + c * kChunk);
        st_stream(m + c * kChunk, v);
      }
      st_stream(out + c * kChunk, v);
    }
  }
}

template <typename T, int BITS, bool STOCH>
__global__ void __launch_bounds__(kThreads) quant_grad_anygroup_kernel(const T* __restrict__ grad, const long long n_groups,
                                                                       uint8_t* __restrict__ packed, float* __restrict__ scales,
                                                                       const unsigned long long seed, const unsigned long long epoch,
                                                                       const Tiling tl, const long long per_cta) {
  overlap_with_neighbours();
  const long long g_lo = (long long)blockIdx.x * per_cta;
  const long long g_hi = g_lo + per_cta < n_groups ? g_lo + per_cta : n_groups;
  quantize_groups<T, BITS, STOCH, false>(tl, grad, nullptr, packed, scales, g_lo, g_hi, seed, epoch, 0xFFFFFFFFu);
}

template <typename T, int BITS>
__global__ void __launch_bounds__(kThreads) dequant_grad_anygroup_kernel(const uint8_t* __restrict__ packed,
                                                                         const float* __restrict__ scales, const long long n_chunks,
                                                                         const int lanes_per_group, T* __restrict__ out) {
  const int lane = threadIdx.x & 31;
  overlap_with_neighbours();
  const long long c = (long long)blockIdx.x * kThreads + threadIdx.x;
  if (c >= n_chunks) return;
  float q[8];
  dequantize8<BITS>(load_codes<BITS>(packed, c, lane, true, false), __ldg(scales + c / lanes_per_group), q);
  st_stream(out + c * kChunk, Conv<T>::pack(q));
}

// grid (CTAs of a sample, samples), every CTA adding its share to the handle's arrival counter
template <typename K, typename Args, typename... Extra>
cudaError_t launch_per_sample(K kernel, const State& st, const Args& a, long long per_cta, cudaStream_t s, Extra... extra) {
  if (a.n_batch <= 0) return cudaSuccess;
  // every CTA's share of the call quantum must be at least 1: very large calls get longer CTAs
  while ((st.groups + per_cta - 1) / per_cta * a.n_batch > (long long)kCallQuantum) per_cta *= 2;
  const long long gx = (st.groups + per_cta - 1) / per_cta;
  const unsigned long long ctas = (unsigned long long)gx * (unsigned long long)a.n_batch;
  LaunchPlan plan = {};
  plan.rows_per_cta = 0;
  plan.share = (unsigned)(kCallQuantum / ctas);
  plan.first_share = (unsigned)(kCallQuantum - (unsigned long long)plan.share * (ctas - 1ull));
  return launch_overlapped(kernel, dim3((unsigned)gx, (unsigned)a.n_batch), s, st, a, plan, extra..., per_cta);
}

}  // namespace

cudaError_t launch_encode_anygroup(int dtype, int bits, const State& st, const EncodeArgs& a, cudaStream_t s) {
  const Tiling tl = tiling_for(st.lanes_per_group);
  const long long per_cta = groups_per_cta(tl);
#define AQ_CALL(T, B)                                                                                         \
  return a.stochastic ? launch_per_sample(encode_anygroup_kernel<T, B, true>, st, a, per_cta, s, tl)          \
                      : launch_per_sample(encode_anygroup_kernel<T, B, false>, st, a, per_cta, s, tl)
  AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
  return cudaErrorInvalidValue;
}

cudaError_t launch_decode_anygroup(int dtype, int bits, const State& st, const DecodeArgs& a, cudaStream_t s) {
  const long long per_cta = groups_per_cta(tiling_for(st.lanes_per_group));
#define AQ_CALL(T, B) return launch_per_sample(decode_anygroup_kernel<T, B>, st, a, per_cta, s, st.lanes_per_group)
  AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
  return cudaErrorInvalidValue;
}

cudaError_t launch_quant_grad_anygroup(int dtype, int bits, int lanes_per_group, const void* grad, long long n_elems,
                                       uint8_t* packed, float* scales, bool stochastic, unsigned long long seed,
                                       unsigned long long epoch, cudaStream_t s) {
  if (n_elems <= 0) return cudaSuccess;
  const Tiling tl = tiling_for(lanes_per_group);
  const long long per_cta = groups_per_cta(tl);
  const long long n_groups = n_elems / kChunk / lanes_per_group;
  const long long grid = (n_groups + per_cta - 1) / per_cta;
  if (grid > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
#define AQ_CALL(T, B)                                                                                                     \
  return stochastic ? launch_overlapped(quant_grad_anygroup_kernel<T, B, true>, dim3((unsigned)grid), s,                 \
                                        reinterpret_cast<const T*>(grad), n_groups, packed, scales, seed, epoch, tl, per_cta) \
                    : launch_overlapped(quant_grad_anygroup_kernel<T, B, false>, dim3((unsigned)grid), s,                \
                                        reinterpret_cast<const T*>(grad), n_groups, packed, scales, seed, epoch, tl, per_cta)
  AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
  return cudaErrorInvalidValue;
}

cudaError_t launch_dequant_grad_anygroup(int dtype, int bits, int lanes_per_group, const uint8_t* packed, const float* scales,
                                         long long n_elems, void* out, cudaStream_t s) {
  if (n_elems <= 0) return cudaSuccess;
  const long long n_chunks = n_elems / kChunk;
  const long long grid = (n_chunks + kThreads - 1) / kThreads;
  if (grid > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
#define AQ_CALL(T, B)                                                                                              \
  return launch_overlapped(dequant_grad_anygroup_kernel<T, B>, dim3((unsigned)grid), s, packed, scales, n_chunks, \
                           lanes_per_group, reinterpret_cast<T*>(out))
  AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
  return cudaErrorInvalidValue;
}

}  // namespace aq
