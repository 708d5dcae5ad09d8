// sm_100a kernels of the AQ-SGD boundary codec: fused encode, fused decode,
// gradient quantize / dequantize, state digest.
//
// The path is bound by HBM traffic (about 6.5 bytes per element), with the issue slots
// of the SMs as the second limit (about 36 thread-instructions per element are available
// at the memory roofline), so the design is about both: every thread moves 128-bit pieces
// ("chunks" of 8 elements of a 2-byte type) with several independent loads in flight, the
// group maximum is a shuffle reduction over the 8 or 16 lanes that hold one group, codes
// leave as whole 32-bit words, m is read and rewritten in place by the same thread in one
// pass, and the quantizer core is written for few instructions (see quantize8).
//
// encode / decode run as several waves of short CTAs on a (rows, samples) grid; each CTA walks
// a few "rows" (256 consecutive chunks) of one sample, so the per-sample work (id lookup,
// first-visit test) is done once per CTA, by its first warp: the kernels have one block
// barrier, at their start, and no wait on another CTA.
//
// Arithmetic: one IEEE binary32 rounding per operation (explicit _rn / _rd intrinsics;
// the one explicit fused multiply-add is exact-equivalent, see quantize8), so the result
// is defined bit for bit.

#include "aq_device.cuh"

namespace aq {
namespace {

// ------------------------------------------------------------------ encode (sender)

// rows that the plain-copy paths (first visit of a sample) move per loop iteration
constexpr int kCopyRows = 4;

// Delta visit of n rows starting at chunk c0 of one sample.  FULL: n == kRowsPerIter and every
// chunk is inside the sample, so no bounds are checked.
template <typename T, int BITS, int LPG, bool STOCH, bool FULL>
__device__ __forceinline__ void encode_rows(const State& st, const EncodeArgs& a, uint32_t stream_id,
                                            const T* __restrict__ act, T* __restrict__ m,
                                            uint8_t* __restrict__ stream, float* __restrict__ scales, int c0,
                                            int n, int lane, bool words_ok) {
  uint4 av[kRowsPerIter], mv[kRowsPerIter];
#pragma unroll
  for (int i = 0; i < kRowsPerIter; ++i) {
    const int c = c0 + i * kThreads;
    if (FULL || (i < n && c < st.chunks)) {
      av[i] = ld_stream(act + (size_t)c * kChunk);
      mv[i] = ld_stream(m + (size_t)c * kChunk);
    } else {
      av[i] = make_uint4(0, 0, 0, 0);
      mv[i] = make_uint4(0, 0, 0, 0);
    }
  }
#pragma unroll
  for (int i = 0; i < kRowsPerIter; ++i) {
    if (FULL || i < n) {                              // uniform over the CTA
      const int c = c0 + i * kThreads;
      const bool active = FULL || c < st.chunks;
      float mf[8], d[8], q[8];
      Conv<T>::unpack(mv[i], mf);
      Conv<T>::diff(av[i], mf, d);
      const float s = group_max<LPG>(abs_max8(d), st.lanes_per_group);
      float delta;
      unsigned long long codes;
      uint4 noise = make_uint4(0, 0, 0, 0);
      if constexpr (STOCH) noise = chunk_noise(a.seed, a.epoch, stream_id, (uint32_t)c);
      quantize8_for<BITS, Conv<T>::kWide, STOCH>(d, s, noise, delta, codes, q);
#pragma unroll
      for (int j = 0; j < 8; ++j) mf[j] = __fadd_rn(mf[j], q[j]);
      if (active) {
        st_stream(m + (size_t)c * kChunk, Conv<T>::pack(mf));
        if ((lane & (st.lanes_per_group - 1)) == 0) scales[c >> st.lg_shift] = delta;
      }
      const bool warp_words = words_ok && (FULL || c - lane + 32 <= st.chunks);
      store_codes<BITS>(stream, c, lane, active, warp_words, codes);
    }
  }
}

// CTAs per multiprocessor that the register budget is cut for: measured, the most that pays
// (the 3-bit kernels spill a few bytes at six and are still 3 % faster than at four; fields
// that straddle words need shuffles and more registers).
template <typename T, int BITS>
constexpr int encode_ctas_per_sm() {
  const bool light = BITS <= 4;                 // codes of a chunk fit one word (3 bits: with a few spilled bytes)
  return !light ? (Conv<T>::kWide ? 3 : 4) : 6;
}
// (The stochastic kernel is bound by instruction issue and gains from every resident warp: six CTAs at 40
// registers with a few spilled bytes ran 4 % faster than four at 64.)
template <int BITS>
constexpr int decode_ctas_per_sm() {
  return (BITS <= 4 || BITS == 8) ? 6 : 4;
}

template <typename T, int BITS, int LPG, bool STOCH>
__global__ void __launch_bounds__(kThreads, STOCH ? (BITS <= 4 ? 6 : 4) : encode_ctas_per_sm<T, BITS>())
    encode_kernel(const State st, const EncodeArgs a, const LaunchPlan plan) {
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int y = blockIdx.y;                                       // sample of the call
  let_dependents_launch();
  // sizes per sample fit 32 bits (checked at create): 32 x 32 -> 64-bit products
  const unsigned elems = (unsigned)st.elems;
  // the sample's buffers: at a fixed stride from the call's base pointers, or (list form) fetched with the sample
  const T* act = reinterpret_cast<const T*>(a.act) + (unsigned long long)(unsigned)y * elems;
  uint8_t* stream = a.packed + (unsigned long long)(unsigned)y * (unsigned)st.packed_bytes;
  float* scales = a.scales + (unsigned long long)(unsigned)y * (unsigned)st.groups;
  // the CTA's chunks [pf_lo, pf_hi): its rows of the activation and of m(xi) are asked for while the
  // previous kernel of the stream is still draining
  const int pf_lo = blockIdx.x * plan.rows_per_cta * kThreads;
  const int pf_hi = min(st.chunks, (int)(blockIdx.x + 1) * plan.rows_per_cta * kThreads);
  if (!STOCH && st.l2_prefetch && tid == 32 && pf_hi > pf_lo) {   // the stochastic kernel is bound by instruction issue
    if (!a.lists) prefetch_l2(act + (size_t)pf_lo * kChunk, (unsigned)(pf_hi - pf_lo) * 16u);
    prefetch_rows_of_m<T>(st, a.ids, y, pf_lo, pf_hi);
  }
  wait_for_predecessor();
  const BufferLists lists = {{a.act_list(), a.packed_list(), a.scales_list(), nullptr}, {true, true, true, false}};
  const Sample sample = open_sample(st, plan, a.ids, y, false, false, a.first_flags, a.lists ? &lists : nullptr);
  const int mode = sample.mode;
  if (a.lists) {
    if (mode == kModeNothing) return;
    act = static_cast<const T*>(sample.buf[0]);
    stream = static_cast<uint8_t*>(const_cast<void*>(sample.buf[1]));
    scales = static_cast<float*>(const_cast<void*>(sample.buf[2]));
  }
  const bool words_ok = (st.packed_bytes & 3) == 0;
  int r = blockIdx.x * plan.rows_per_cta;                         // this CTA's rows of the sample: [r, r_end)
  const int r_end = min(st.rows, r + plan.rows_per_cta);

  if (mode == kModeDelta) {
    T* m = reinterpret_cast<T*>(st.m) + (unsigned long long)sample.row * elems;
    // whole iterations first (rows without a ragged end: no bounds to check), then the rest
    const int whole_end = min(r_end, st.chunks / kThreads);
    for (; r + kRowsPerIter <= whole_end; r += kRowsPerIter)
      encode_rows<T, BITS, LPG, STOCH, true>(st, a, (uint32_t)sample.id, act, m, stream, scales, r * kThreads + tid,
                                             kRowsPerIter, lane, words_ok);
    for (; r < r_end; r += kRowsPerIter)
      encode_rows<T, BITS, LPG, STOCH, false>(st, a, (uint32_t)sample.id, act, m, stream, scales, r * kThreads + tid,
                                              min(kRowsPerIter, r_end - r), lane, words_ok);
  } else {
    // first visit: the activation itself becomes m(xi); skipped sample: nothing is stored.
    // Either way the sample's codes and scales are zero.
    T* m = (mode == kModeFirst) ? reinterpret_cast<T*>(st.m) + (unsigned long long)sample.row * elems : nullptr;
    // kCopyRows rows at a time, their loads in flight together before the first store
    for (; r < r_end; r += kCopyRows) {
      uint4 v[kCopyRows];
#pragma unroll
      for (int i = 0; i < kCopyRows; ++i) {
        const int c = (r + i) * kThreads + tid;
        v[i] = make_uint4(0, 0, 0, 0);
        if (m && r + i < r_end && c < st.chunks) v[i] = ld_stream(act + (size_t)c * kChunk);
      }
#pragma unroll
      for (int i = 0; i < kCopyRows; ++i) {
        if (r + i < r_end) {                          // uniform over the CTA
          const int c = (r + i) * kThreads + tid;
          const bool active = c < st.chunks;
          if (active) {
            if (m) st_stream(m + (size_t)c * kChunk, v[i]);
            if ((lane & (st.lanes_per_group - 1)) == 0) scales[c >> st.lg_shift] = 0.0f;
          }
          const bool warp_words = words_ok && (c - lane + 32 <= st.chunks);
          store_codes<BITS>(stream, c, lane, active, warp_words, 0ull);
        }
      }
    }
  }
}

// ------------------------------------------------------------------ decode (receiver)

template <typename T, int BITS, bool FULL>
__device__ __forceinline__ void decode_rows(const State& st, const uint8_t* __restrict__ stream,
                                            const float* __restrict__ scales, T* __restrict__ m,
                                            T* __restrict__ out, int c0, int n, int lane, bool words_ok) {
  uint4 mv[kRowsPerIter];
  unsigned long long codes[kRowsPerIter];
  float delta[kRowsPerIter];
#pragma unroll
  for (int i = 0; i < kRowsPerIter; ++i) {
    const int c = c0 + i * kThreads;
    const bool active = FULL || (i < n && c < st.chunks);
    if (active) {
      mv[i] = ld_stream(m + (size_t)c * kChunk);
      delta[i] = __ldg(scales + (c >> st.lg_shift));
    } else {
      mv[i] = make_uint4(0, 0, 0, 0);
      delta[i] = 0.0f;
    }
    codes[i] = 0ull;
    if (FULL || i < n) {                              // uniform over the CTA
      const bool warp_words = words_ok && (FULL || c - lane + 32 <= st.chunks);
      codes[i] = load_codes<BITS>(stream, c, lane, active, warp_words);
    }
  }
#pragma unroll
  for (int i = 0; i < kRowsPerIter; ++i) {
    const int c = c0 + i * kThreads;
    if (FULL || (i < n && c < st.chunks)) {
      float mf[8], q[8];
      Conv<T>::unpack(mv[i], mf);
      dequantize8<BITS>(codes[i], delta[i], q);
#pragma unroll
      for (int j = 0; j < 8; ++j) mf[j] = __fadd_rn(mf[j], q[j]);
      const uint4 nv = Conv<T>::pack(mf);
      st_stream(m + (size_t)c * kChunk, nv);
      st_stream(out + (size_t)c * kChunk, nv);
    }
  }
}

// LISTS: the call names its buffers through arrays of pointers (a.lists); an instantiation of its own,
// so that the base-pointer form keeps its addresses in closed form.
template <typename T, int BITS, bool LISTS>
__global__ void __launch_bounds__(kThreads, decode_ctas_per_sm<BITS>()) decode_kernel(const State st, const DecodeArgs a, const LaunchPlan plan) {
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const CtaRows cta = locate_cta(plan);
  const int y = cta.y;                                            // sample of the call
  let_dependents_launch();
  int r = cta.x * cta.rows;                                       // this CTA's rows of the sample: [r, r_end)
  const int r_end = min(st.rows, r + cta.rows);
  // the CTA's rows of m(xi) are asked for while the previous kernel of the stream is still draining
  if (st.l2_prefetch && tid == 32) prefetch_rows_of_m<T>(st, a.ids, y, r * kThreads, min(st.chunks, r_end * kThreads));
  wait_for_predecessor();
  const BufferLists lists = {{a.packed_list(), a.scales_list(), a.raw_list(), a.out_list()}, {true, true, false, true}};
  const Sample sample = open_sample(st, plan, a.ids, y, true, a.raw != nullptr, a.first_flags, LISTS ? &lists : nullptr,
                                    a.raw != nullptr ? 2 : -1, cta.x);
  const int mode = sample.mode;
  const unsigned elems = (unsigned)st.elems;
  // the sample's buffers: at a fixed stride from the call's base pointers, or (list form) fetched with the sample
  T* out = reinterpret_cast<T*>(a.out) + (unsigned long long)(unsigned)y * elems;
  const uint8_t* stream = a.packed + (unsigned long long)(unsigned)y * (unsigned)st.packed_bytes;
  const float* scales = a.scales + (unsigned long long)(unsigned)y * (unsigned)st.groups;
  const T* raw = a.raw ? reinterpret_cast<const T*>(a.raw) + (unsigned long long)(unsigned)y * elems : nullptr;
  if constexpr (LISTS) {
    if (mode == kModeNothing) return;
    stream = static_cast<const uint8_t*>(sample.buf[0]);
    scales = static_cast<const float*>(sample.buf[1]);
    raw = static_cast<const T*>(sample.buf[2]);
    out = static_cast<T*>(const_cast<void*>(sample.buf[3]));
  }

  if (mode == kModeDelta) {
    T* m = reinterpret_cast<T*>(st.m) + (unsigned long long)sample.row * elems;
    const bool words_ok = (st.packed_bytes & 3) == 0;
    const int whole_end = min(r_end, st.chunks / kThreads);
    for (; r + kRowsPerIter <= whole_end; r += kRowsPerIter)
      decode_rows<T, BITS, true>(st, stream, scales, m, out, r * kThreads + tid, kRowsPerIter, lane, words_ok);
    for (; r < r_end; r += kRowsPerIter)
      decode_rows<T, BITS, false>(st, stream, scales, m, out, r * kThreads + tid, min(kRowsPerIter, r_end - r), lane,
                                  words_ok);
  } else {
    // first visit: the raw message becomes m(xi) and the activation; skipped sample: zeros out.
    const bool first = mode == kModeFirst;
    T* m = first ? reinterpret_cast<T*>(st.m) + (unsigned long long)sample.row * elems : nullptr;
    for (; r < r_end; r += kCopyRows) {
      uint4 v[kCopyRows];
#pragma unroll
      for (int i = 0; i < kCopyRows; ++i) {
        const int c = (r + i) * kThreads + tid;
        v[i] = make_uint4(0, 0, 0, 0);
        if (first && r + i < r_end && c < st.chunks) v[i] = ld_stream(raw + (size_t)c * kChunk);
      }
#pragma unroll
      for (int i = 0; i < kCopyRows; ++i) {
        const int c = (r + i) * kThreads + tid;
        if (r + i < r_end && c < st.chunks) {
          if (first) st_stream(m + (size_t)c * kChunk, v[i]);
          st_stream(out + (size_t)c * kChunk, v[i]);
        }
      }
    }
  }
}

// ------------------------------------------------------------------ backward direction: direct quantization

template <typename T, int BITS, int LPG, bool STOCH>
__global__ void __launch_bounds__(kThreads) quant_grad_kernel(const T* __restrict__ grad, long long n_chunks,
                                                              int lanes_per_group, uint8_t* __restrict__ packed,
                                                              float* __restrict__ scales, unsigned long long seed,
                                                              unsigned long long epoch, int l2_prefetch) {
  const int lane = threadIdx.x & 31;
  const int lg_shift = __ffs(lanes_per_group) - 1;
  const long long c0 = (long long)blockIdx.x * kChunksPerCta + threadIdx.x;
  let_dependents_launch();
  if (l2_prefetch && threadIdx.x == 0) {            // the CTA's piece of the gradient, asked for while the previous kernel drains
    const long long lo = (long long)blockIdx.x * kChunksPerCta;
    const long long hi = lo + kChunksPerCta < n_chunks ? lo + kChunksPerCta : n_chunks;
    if (hi > lo) prefetch_l2(grad + lo * kChunk, (unsigned)(hi - lo) * 16u);
  }
  wait_for_predecessor();
  uint4 gv[kChunksPerThread];
#pragma unroll
  for (int i = 0; i < kChunksPerThread; ++i) {
    const long long c = c0 + i * kThreads;
    gv[i] = (c < n_chunks) ? ld_stream(grad + c * kChunk) : make_uint4(0, 0, 0, 0);
  }
#pragma unroll
  for (int i = 0; i < kChunksPerThread; ++i) {
    const long long c = c0 + i * kThreads;
    const bool active = c < n_chunks;
    float d[8], q[8];
    Conv<T>::unpack(gv[i], d);
    const float s = group_max<LPG>(abs_max8(d), lanes_per_group);
    float delta;
    unsigned long long codes;
    uint4 noise = make_uint4(0, 0, 0, 0);
    if constexpr (STOCH) noise = chunk_noise(seed, epoch, 0xFFFFFFFFu, (uint32_t)c);
    quantize8_for<BITS, Conv<T>::kWide, STOCH>(d, s, noise, delta, codes, q);
    if (active && (lane & (lanes_per_group - 1)) == 0) scales[c >> lg_shift] = delta;
    store_codes<BITS>(packed, c, lane, active, c - lane + 32 <= n_chunks, codes);
  }
}

// Chunks are numbered with 32 bits inside a launch (the launch layer cuts longer inputs into slices), and
// a CTA whose chunks all exist takes a path without bounds: with two bytes written per element and less
// than one read, this kernel has few loads to wait for and is bound by its instruction count.
template <typename T, int BITS, bool FULL>
__device__ __forceinline__ void dequant_chunks(const uint8_t* __restrict__ packed, const float* __restrict__ scales,
                                               unsigned n_chunks, int lg_shift, T* __restrict__ out, unsigned c0, int lane) {
  unsigned long long codes[kChunksPerThread];
  float delta[kChunksPerThread];
#pragma unroll
  for (int i = 0; i < kChunksPerThread; ++i) {
    const unsigned c = c0 + i * kThreads;
    const bool active = FULL || c < n_chunks;
    delta[i] = active ? __ldg(scales + (c >> lg_shift)) : 0.0f;
    codes[i] = load_codes<BITS>(packed, c, lane, active, FULL || c - lane + 32 <= n_chunks);
  }
#pragma unroll
  for (int i = 0; i < kChunksPerThread; ++i) {
    const unsigned c = c0 + i * kThreads;
    if (FULL || c < n_chunks) {
      float q[8];
      dequantize8<BITS>(codes[i], delta[i], q);
      st_stream(out + (size_t)c * kChunk, Conv<T>::pack(q));
    }
  }
}

template <typename T, int BITS>
__global__ void __launch_bounds__(kThreads) dequant_grad_kernel(const uint8_t* __restrict__ packed,
                                                                const float* __restrict__ scales, unsigned n_chunks,
                                                                int lg_shift, T* __restrict__ out) {
  const int lane = threadIdx.x & 31;
  const unsigned c0 = blockIdx.x * (unsigned)kChunksPerCta + threadIdx.x;
  overlap_with_neighbours();
  if ((blockIdx.x + 1) * (unsigned)kChunksPerCta <= n_chunks)
    dequant_chunks<T, BITS, true>(packed, scales, n_chunks, lg_shift, out, c0, lane);
  else
    dequant_chunks<T, BITS, false>(packed, scales, n_chunks, lg_shift, out, c0, lane);
}

// ---- quantization with sixteen elements per lane
// A lane owns two neighbouring chunks (32 contiguous bytes of the gradient).  A group of 64 is
// then 4 lanes instead of 8 (two shuffle steps for its maximum instead of three, one reciprocal
// per 16 elements instead of per 8), and the codes of a lane are whole words for every width
// but 3 (6 bits: 96 bits = three words; 3 bits: two lanes share three words), so no code crosses
// a lane.  Built for 1, 2, 3, 4, 6 and 8 bits and groups of 16 elements or more; the one-chunk
// kernel above takes the rest.  (Loads of 16 bytes at a 32-byte stride are merged in L1; the
// same shape on the way out -- two half-sector stores per lane -- measured slower than the dense
// stores of dequant_grad_kernel, so the inverse keeps one chunk per lane.)

constexpr int kPairsPerThread = 2;
constexpr int kPairsPerCta = kThreads * kPairsPerThread;

__host__ __device__ constexpr bool wide_lane_bits(int bits) { return bits == 1 || bits == 2 || bits == 3 || bits == 4 || bits == 6 || bits == 8; }

// Codes of 16 elements (c0: the first chunk, c1: the second) to their place in the stream.
template <int BITS>
__device__ __forceinline__ void store_codes16(uint8_t* stream, long long pair, int lane, bool active, bool partner_active,
                                              unsigned long long c0, unsigned long long c1) {
  if constexpr (BITS == 8) {
    if (active) *reinterpret_cast<uint4*>(stream + pair * 16) = make_uint4((unsigned)c0, (unsigned)(c0 >> 32), (unsigned)c1, (unsigned)(c1 >> 32));
  } else if constexpr (BITS == 4) {
    if (active) *reinterpret_cast<uint2*>(stream + pair * 8) = make_uint2((unsigned)c0, (unsigned)c1);
  } else if constexpr (BITS == 2) {
    if (active) *reinterpret_cast<uint32_t*>(stream + pair * 4) = (uint32_t)c0 | ((uint32_t)c1 << 16);
  } else if constexpr (BITS == 1) {
    if (active) *reinterpret_cast<uint16_t*>(stream + pair * 2) = (uint16_t)((uint32_t)c0 | ((uint32_t)c1 << 8));
  } else if constexpr (BITS == 6) {
    if (active) {
      uint32_t* w = reinterpret_cast<uint32_t*>(stream + pair * 12);
      w[0] = (uint32_t)c0;
      w[1] = (uint32_t)(c0 >> 32) | ((uint32_t)c1 << 16);
      w[2] = (uint32_t)(c1 >> 16);
    }
  } else {
    static_assert(BITS == 3, "no sixteen-element form for this width");
    // 48 bits per lane; an even lane and the next one share three words
    const uint32_t lo = (uint32_t)c0 | ((uint32_t)c1 << 24), hi = (uint32_t)c1 >> 8;      // bits [0,32) and [32,48)
    const uint32_t other = __shfl_xor_sync(kFullMask, lo, 1);
    const bool odd = lane & 1;
    uint8_t* base = stream + (pair >> 1) * 12;
    if (active) {
      if (odd) {
        *reinterpret_cast<uint32_t*>(base + 8) = (lo >> 16) | (hi << 16);
      } else {
        *reinterpret_cast<uint32_t*>(base) = lo;
        if (partner_active) *reinterpret_cast<uint32_t*>(base + 4) = hi | (other << 16);
        else *reinterpret_cast<uint16_t*>(base + 4) = (uint16_t)hi;                        // the stream ends with this lane
      }
    }
  }
}

template <typename T, int BITS, int LPG, bool STOCH>
__global__ void __launch_bounds__(kThreads) quant_grad16_kernel(const T* __restrict__ grad, long long n_pairs,
                                                                int lanes_per_group, uint8_t* __restrict__ packed,
                                                                float* __restrict__ scales, unsigned long long seed,
                                                                unsigned long long epoch, int l2_prefetch) {
  const int lane = threadIdx.x & 31;
  const int lg_shift = __ffs(lanes_per_group) - 1;
  const long long p0 = (long long)blockIdx.x * kPairsPerCta + threadIdx.x;
  let_dependents_launch();
  if (l2_prefetch && threadIdx.x == 0) {            // the CTA's piece of the gradient, asked for while the previous kernel drains
    const long long lo = (long long)blockIdx.x * kPairsPerCta;
    const long long hi = lo + kPairsPerCta < n_pairs ? lo + kPairsPerCta : n_pairs;
    if (hi > lo) prefetch_l2(grad + lo * 2 * kChunk, (unsigned)(hi - lo) * 32u);
  }
  wait_for_predecessor();
  uint4 gv[kPairsPerThread][2];
#pragma unroll
  for (int i = 0; i < kPairsPerThread; ++i) {
    const long long p = p0 + i * kThreads;
    const bool active = p < n_pairs;
    gv[i][0] = active ? ld_stream(grad + p * 2 * kChunk) : make_uint4(0, 0, 0, 0);
    gv[i][1] = active ? ld_stream(grad + p * 2 * kChunk + kChunk) : make_uint4(0, 0, 0, 0);
  }
#pragma unroll
  for (int i = 0; i < kPairsPerThread; ++i) {
    const long long p = p0 + i * kThreads;
    const bool active = p < n_pairs;
    float d0[8], d1[8], q[8];
    Conv<T>::unpack(gv[i][0], d0);
    Conv<T>::unpack(gv[i][1], d1);
    const float s = group_max<LPG>(fmaxf(abs_max8(d0), abs_max8(d1)), lanes_per_group);
    float delta;
    unsigned long long c0, c1;
    uint4 n0 = make_uint4(0, 0, 0, 0), n1 = make_uint4(0, 0, 0, 0);
    if constexpr (STOCH) {
      n0 = chunk_noise(seed, epoch, 0xFFFFFFFFu, (uint32_t)(2 * p));
      n1 = chunk_noise(seed, epoch, 0xFFFFFFFFu, (uint32_t)(2 * p + 1));
    }
    quantize8_for<BITS, Conv<T>::kWide, STOCH>(d0, s, n0, delta, c0, q);
    quantize8_for<BITS, Conv<T>::kWide, STOCH>(d1, s, n1, delta, c1, q);
    if (active && (lane & (lanes_per_group - 1)) == 0) scales[p >> lg_shift] = delta;
    store_codes16<BITS>(packed, p, lane, active, p + 1 < n_pairs, c0, c1);
  }
}

// ------------------------------------------------------------------ rows between a store and a staging block

constexpr int kCopyPiecesPerThread = 4;

template <typename Piece>
__global__ void __launch_bounds__(kThreads) copy_rows_kernel(const Piece* __restrict__ src, Piece* __restrict__ dst,
                                                             const int32_t* __restrict__ ids, long long row_pieces,
                                                             bool gather) {
  const int y = blockIdx.y;
  const long long id = ids[y];
  if (id < 0) return;
  const Piece* from = src + (gather ? id : (long long)y) * row_pieces;
  Piece* to = dst + (gather ? (long long)y : id) * row_pieces;
  const long long p0 = (long long)blockIdx.x * (kThreads * kCopyPiecesPerThread) + threadIdx.x;
  Piece v[kCopyPiecesPerThread];
#pragma unroll
  for (int i = 0; i < kCopyPiecesPerThread; ++i) {
    const long long p = p0 + i * kThreads;
    if (p < row_pieces) v[i] = from[p];
  }
#pragma unroll
  for (int i = 0; i < kCopyPiecesPerThread; ++i) {
    const long long p = p0 + i * kThreads;
    if (p < row_pieces) to[p] = v[i];
  }
}

// ------------------------------------------------------------------ the wire between two stages on one device

constexpr int kWirePiecesPerThread = 4;

// Up to three byte ranges copied by one launch (codes, steps and, on first visits, the raw block):
// range k holds n[k] 16-byte pieces; the grid walks the ranges laid end to end.  Overlapped with its
// neighbours in the stream like the codec kernels, so a copy between encode and decode costs one
// launch instead of one per buffer.
struct WireRanges {
  const uint4* src[3];
  uint4* dst[3];
  long long n[3];
};

__global__ void __launch_bounds__(kThreads) wire_copy_kernel(const WireRanges w) {
  overlap_with_neighbours();
  const long long total = w.n[0] + w.n[1] + w.n[2];
  const long long p0 = (long long)blockIdx.x * (kThreads * kWirePiecesPerThread) + threadIdx.x;
  uint4 v[kWirePiecesPerThread];
  int which[kWirePiecesPerThread];
  long long at[kWirePiecesPerThread];
#pragma unroll
  for (int i = 0; i < kWirePiecesPerThread; ++i) {
    long long p = p0 + i * kThreads;
    which[i] = -1;
    if (p < total) {
      int k = 0;
      if (p >= w.n[0]) { p -= w.n[0]; k = 1; }
      if (k == 1 && p >= w.n[1]) { p -= w.n[1]; k = 2; }
      which[i] = k;
      at[i] = p;
      v[i] = w.src[k][p];
    }
  }
#pragma unroll
  for (int i = 0; i < kWirePiecesPerThread; ++i)
    if (which[i] >= 0) w.dst[which[i]][at[i]] = v[i];
}

// ------------------------------------------------------------------ state digest

__device__ __forceinline__ unsigned long long mix64(unsigned long long index, unsigned long long word) {
  unsigned long long z = index * 0x9E3779B97F4A7C15ull + word;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

__global__ void __launch_bounds__(kThreads) checksum_kernel(const State st, unsigned long long* sum_out) {
  const long long n_vec = st.n_samples * (long long)st.chunks;      // 16-byte pieces = two 64-bit words each
  const uint4* mv = reinterpret_cast<const uint4*>(st.m);
  const long long stride = (long long)gridDim.x * kThreads;
  unsigned long long acc = 0ull;
  for (long long v = (long long)blockIdx.x * kThreads + threadIdx.x; v < n_vec; v += stride) {
    const uint4 w = __ldcs(mv + v);
    const unsigned long long i = (unsigned long long)v * 2ull;
    acc += mix64(i, ((unsigned long long)w.y << 32) | w.x) + mix64(i + 1, ((unsigned long long)w.w << 32) | w.z);
  }
  for (long long x = (long long)blockIdx.x * kThreads + threadIdx.x; x < st.n_samples; x += stride)
    acc += mix64((1ull << 40) + (unsigned long long)x, st.seen[x] != 0ull ? 1ull : 0ull);
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(kFullMask, acc, o);
  __shared__ unsigned long long part[kThreads / 32];
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long t = 0ull;
    for (int w = 0; w < kThreads / 32; ++w) t += part[w];
    atomicAdd(sum_out, t);
  }
}

__global__ void __launch_bounds__(kThreads) checksum_lowbit_kernel(const State st, unsigned long long* sum_out) {
  const long long n_code_words = st.n_samples * st.m_bytes / 4;      // the code bytes of all samples as one array
  const long long n_scale_words = st.m_scales ? st.n_samples * st.groups : 0;
  const uint32_t* cw = static_cast<const uint32_t*>(st.m);
  const uint32_t* sw = reinterpret_cast<const uint32_t*>(st.m_scales);
  const long long stride = (long long)gridDim.x * kThreads;
  const long long first = (long long)blockIdx.x * kThreads + threadIdx.x;
  unsigned long long acc = 0ull;
  for (long long i = first; i < n_code_words; i += stride) acc += mix64((unsigned long long)i, cw[i]);
  for (long long i = first; i < n_scale_words; i += stride) acc += mix64((unsigned long long)(n_code_words + i), sw[i]);
  for (long long x = first; x < st.n_samples; x += stride)
    acc += mix64((1ull << 40) + (unsigned long long)x, st.seen[x] != 0ull ? 1ull : 0ull);
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(kFullMask, acc, o);
  __shared__ unsigned long long part[kThreads / 32];
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long t = 0ull;
    for (int w = 0; w < kThreads / 32; ++w) t += part[w];
    atomicAdd(sum_out, t);
  }
}

template <typename T, int BITS>
cudaError_t launch_quant16(int lanes16, const void* grad, long long pairs, uint8_t* packed, float* scales, bool stochastic,
                           unsigned long long seed, unsigned long long epoch, int l2_prefetch, cudaStream_t s) {
  if constexpr (wide_lane_bits(BITS)) {
    const dim3 grid((unsigned)((pairs + kPairsPerCta - 1) / kPairsPerCta));
    const T* g = reinterpret_cast<const T*>(grad);
#define AQ_CALL_LPG16(L)                                                                                                           \
  return stochastic ? launch_overlapped(quant_grad16_kernel<T, BITS, L, true>, grid, s, g, pairs, lanes16, packed, scales, seed, epoch, 0) \
                    : launch_overlapped(quant_grad16_kernel<T, BITS, L, false>, grid, s, g, pairs, lanes16, packed, scales, seed, epoch, l2_prefetch)
    switch (lanes16) {
      case 4: AQ_CALL_LPG16(4);
      case 8: AQ_CALL_LPG16(8);
      default: AQ_CALL_LPG16(0);
    }
#undef AQ_CALL_LPG16
  } else {
    return cudaErrorInvalidValue;
  }
}

inline unsigned grid_x(long long chunks) { return (unsigned)((chunks + kChunksPerCta - 1) / kChunksPerCta); }

// Rows per CTA and CTAs per sample of an encode / decode launch.
struct RowSplit {
  long long per, gx;
};
inline RowSplit split_rows(const State& st, int n_batch) {
  const long long total = (long long)n_batch * st.rows;
  long long per = st.rows_per_cta;
  if (per <= 0) {
    // a small call gets the fewest rows per CTA that still put the whole grid on the multiprocessors at once
    // (six CTAs each): one sequence of 800 rows runs as 800 CTAs of one row, measured 3.7 us per call against
    // 4.2 us at two rows and 6.4 us at four; large calls take kRowsPerCta
    const long long slots = (long long)st.sms * 6;
    per = (total + slots - 1) / slots;
    per = per < 1 ? 1 : (per > kRowsPerCta ? kRowsPerCta : per);
  }
  if (per > st.rows) per = st.rows;
  long long gx = (st.rows + per - 1) / per;
  if (gx * n_batch > (long long)kCallQuantum) {            // keep every CTA's share of the quantum >= 1
    gx = (long long)kCallQuantum / n_batch;
    per = (st.rows + gx - 1) / gx;
    gx = (st.rows + per - 1) / per;
  }
  return {per, gx};
}

inline void set_shares(LaunchPlan& plan, unsigned long long ctas) {
  plan.share = (unsigned)(kCallQuantum / ctas);
  plan.first_share = (unsigned)(kCallQuantum - (unsigned long long)plan.share * (ctas - 1ull));
}

// Grid (CTAs of a sample, samples).
template <typename K, typename Args>
cudaError_t launch_rows(K kernel, const State& st, const Args& a, cudaStream_t s) {
  if (a.n_batch <= 0) return cudaSuccess;
  const RowSplit sp = split_rows(st, a.n_batch);
  LaunchPlan plan = {};
  plan.rows_per_cta = (int)sp.per;
  set_shares(plan, (unsigned long long)sp.gx * (unsigned long long)a.n_batch);
  return launch_overlapped(kernel, dim3((unsigned)sp.gx, (unsigned)a.n_batch), s, st, a, plan);
}

// One-dimensional grid in the same order (the CTAs of sample 0, then those of sample 1, ...) whose end tapers:
// when a grid runs out of CTAs, every multiprocessor still has to finish the ones it holds, and how long that
// takes is set by the rows a CTA walks.  On a call of several waves of full-size CTAs the last samples -- about
// one wave of the resident CTA slots at half the rows -- are therefore walked by CTAs of half the rows.
template <typename K, typename Args>
cudaError_t launch_rows_tapered(K kernel, const State& st, const Args& a, cudaStream_t s) {
  if (a.n_batch <= 0) return cudaSuccess;
  const RowSplit sp = split_rows(st, a.n_batch);
  const long long slots = (long long)st.sms * 6;
  long long tail_rows = sp.per, gx2 = sp.gx;
  int n2 = 0;
  if (st.rows_per_cta <= 0 && sp.per == kRowsPerCta && sp.gx * a.n_batch >= 2 * slots) {
    tail_rows = sp.per / 2;
    gx2 = (st.rows + tail_rows - 1) / tail_rows;
    n2 = (int)(slots * tail_rows / st.rows);
    n2 = n2 < 1 ? 1 : n2;
    if (n2 > a.n_batch / 2) n2 = a.n_batch / 2;
  }
  const int n1 = a.n_batch - n2;
  const unsigned long long ctas = (unsigned long long)sp.gx * n1 + (unsigned long long)gx2 * n2;
  LaunchPlan plan = {};
  plan.rows_per_cta = (int)sp.per;
  plan.ctas1 = (unsigned)(sp.gx * n1);
  plan.gx1 = (unsigned)sp.gx;
  plan.gx2 = (unsigned)gx2;
  plan.n1 = n1;
  plan.tail_rows = (int)tail_rows;
  if (ctas > kCallQuantum) {                               // no taper: split_rows has bounded gx * n_batch
    plan.ctas1 = (unsigned)(sp.gx * a.n_batch);
    plan.n1 = a.n_batch;
    set_shares(plan, plan.ctas1);
    return launch_overlapped(kernel, dim3(plan.ctas1), s, st, a, plan);
  }
  set_shares(plan, ctas);
  return launch_overlapped(kernel, dim3((unsigned)ctas), s, st, a, plan);
}

}  // namespace

cudaError_t launch_encode(int dtype, int bits, const State& st, const EncodeArgs& a, cudaStream_t s) {
#define AQ_CALL_LPG(L)                                                         \
  return a.stochastic ? launch_rows(encode_kernel<T_, B_, L, true>, st, a, s) \
                      : launch_rows(encode_kernel<T_, B_, L, false>, st, a, s)
#define AQ_CALL(T, B)                                      \
  {                                                        \
    using T_ = T;                                          \
    constexpr int B_ = B;                                  \
    AQ_WITH_LPG(st.lanes_per_group, AQ_CALL_LPG)           \
  }
  AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
#undef AQ_CALL_LPG
  return cudaErrorInvalidValue;
}

cudaError_t launch_decode(int dtype, int bits, const State& st, const DecodeArgs& a, cudaStream_t s) {
#define AQ_CALL(T, B) return a.lists ? launch_rows_tapered(decode_kernel<T, B, true>, st, a, s) : launch_rows_tapered(decode_kernel<T, B, false>, st, a, s)
  AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
  return cudaErrorInvalidValue;
}

cudaError_t launch_quant_grad(int dtype, int bits, int lanes_per_group, const void* grad, long long n_elems,
                              uint8_t* packed, float* scales, bool stochastic, unsigned long long seed,
                              unsigned long long epoch, int l2_prefetch, cudaStream_t s) {
  if (n_elems <= 0) return cudaSuccess;
  const long long chunks = n_elems / kChunk;
  if (wide_lane_bits(bits) && lanes_per_group >= 2) {             // sixteen elements per lane
#define AQ_CALL16(T, B) return launch_quant16<T, B>(lanes_per_group / 2, grad, chunks / 2, packed, scales, stochastic, seed, epoch, l2_prefetch, s)
    AQ_DISPATCH(dtype, bits, AQ_CALL16)
#undef AQ_CALL16
  }
  const unsigned grid = grid_x(chunks);
#define AQ_CALL_LPG(L)                                                                                              \
  return stochastic ? launch_overlapped(quant_grad_kernel<T_, B_, L, true>, dim3(grid), s,                          \
                                        reinterpret_cast<const T_*>(grad), chunks, lanes_per_group, packed, scales, \
                                        seed, epoch, 0)                                                             \
                    : launch_overlapped(quant_grad_kernel<T_, B_, L, false>, dim3(grid), s,                         \
                                        reinterpret_cast<const T_*>(grad), chunks, lanes_per_group, packed, scales, \
                                        seed, epoch, l2_prefetch)
#define AQ_CALL(T, B)                                      \
  {                                                        \
    using T_ = T;                                          \
    constexpr int B_ = B;                                  \
    AQ_WITH_LPG(lanes_per_group, AQ_CALL_LPG)              \
  }
  AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
#undef AQ_CALL_LPG
  return cudaGetLastError();
}

cudaError_t launch_dequant_grad(int dtype, int bits, int lanes_per_group, const uint8_t* packed, const float* scales,
                                long long n_elems, void* out, cudaStream_t s) {
  if (n_elems <= 0) return cudaSuccess;
  int lg_shift = 0;
  while ((1 << lg_shift) < lanes_per_group) ++lg_shift;
  // slices of at most 2^27 chunks (byte offsets into the codes then fit 32 bits), each a multiple of a CTA's
  // chunks and therefore of a group and a warp
  const long long slice = (1ll << 27) / kChunksPerCta * kChunksPerCta;
  for (long long done = 0, chunks = n_elems / kChunk; done < chunks; done += slice) {
    const unsigned n = (unsigned)(chunks - done < slice ? chunks - done : slice);
    const uint8_t* p = packed + done * bits;
    const float* sc = scales + (done >> lg_shift);
    cudaError_t e = cudaErrorInvalidValue;
#define AQ_CALL(T, B)                                                                                             \
  e = launch_overlapped(dequant_grad_kernel<T, B>, dim3(grid_x(n)), s, p, sc, n, lg_shift, reinterpret_cast<T*>(out) + done * kChunk); \
  break
    AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

cudaError_t launch_copy_rows(const void* src, void* dst, const int32_t* ids, int n, long long row_bytes, bool gather,
                             cudaStream_t s) {
  if (n <= 0 || row_bytes <= 0) return cudaSuccess;
  const long long per_cta = (long long)kThreads * kCopyPiecesPerThread;
  // the widest piece that divides a row and that both blocks are aligned for
  const uintptr_t where = reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst) | (uintptr_t)row_bytes;
  const int piece = (where & 15u) == 0 ? 16 : (where & 3u) == 0 ? 4 : 1;
  const long long pieces = row_bytes / piece;
  const dim3 grid((unsigned)((pieces + per_cta - 1) / per_cta), (unsigned)n);
  if (piece == 16)
    copy_rows_kernel<uint4><<<grid, kThreads, 0, s>>>(static_cast<const uint4*>(src), static_cast<uint4*>(dst), ids, pieces, gather);
  else if (piece == 4)
    copy_rows_kernel<uint32_t><<<grid, kThreads, 0, s>>>(static_cast<const uint32_t*>(src), static_cast<uint32_t*>(dst), ids, pieces,
                                                         gather);
  else
    copy_rows_kernel<uint8_t><<<grid, kThreads, 0, s>>>(static_cast<const uint8_t*>(src), static_cast<uint8_t*>(dst), ids, pieces,
                                                        gather);
  return cudaGetLastError();
}

cudaError_t launch_wire_copy(const void* const* src, void* const* dst, const size_t* bytes, int n_ranges, cudaStream_t s) {
  WireRanges w = {};
  long long total = 0;
  for (int k = 0; k < n_ranges && k < 3; ++k) {
    w.src[k] = static_cast<const uint4*>(src[k]);
    w.dst[k] = static_cast<uint4*>(dst[k]);
    w.n[k] = (long long)(bytes[k] / 16);
    total += w.n[k];
  }
  if (total == 0) return cudaSuccess;
  const long long per_cta = (long long)kThreads * kWirePiecesPerThread;
  return launch_overlapped(wire_copy_kernel, dim3((unsigned)((total + per_cta - 1) / per_cta)), s, w);
}

cudaError_t launch_checksum(const State& st, unsigned long long* sum_dev, cudaStream_t s) {
  if (st.m_bits) {
    const long long words = st.n_samples * st.m_bytes / 4;
    long long want = (words + kThreads - 1) / kThreads;
    const long long cap = (long long)st.sms * 8;
    checksum_lowbit_kernel<<<(unsigned)(want < 1 ? 1 : (want > cap ? cap : want)), kThreads, 0, s>>>(st, sum_dev);
    return cudaGetLastError();
  }
  const long long n_vec = st.n_samples * (long long)st.chunks;
  long long want = (n_vec + kThreads - 1) / kThreads;
  const long long cap = (long long)st.sms * 8;
  const unsigned grid = (unsigned)(want < 1 ? 1 : (want > cap ? cap : want));
  checksum_kernel<<<grid, kThreads, 0, s>>>(st, sum_dev);
  return cudaGetLastError();
}

}  // namespace aq
