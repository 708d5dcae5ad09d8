// sm_100a kernels of the AQ-SGD boundary codec: fused encode, fused decode,
// gradient quantize / dequantize, state digest.
//
// The path is bound by HBM traffic (about 6.5 bytes per element against roughly
// 20 arithmetic instructions), so the design is about memory: every thread moves
// 128-bit pieces ("chunks" of 8 elements of a 2-byte type) with several
// independent loads in flight, the group maximum is a shuffle reduction over the
// 8 or 16 lanes that hold one group, codes leave as whole 32-bit words, and m is
// read and rewritten in place by the same thread in one pass.
//
// Arithmetic: one IEEE binary32 rounding per operation (explicit _rn / _rd
// intrinsics, never contracted into a fused multiply-add), so the result is
// defined bit for bit.

#include "aq_internal.h"

#include <cfloat>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

namespace aq {
namespace {

constexpr unsigned kFullMask = 0xffffffffu;
constexpr int kChunksPerCta = kThreads * kChunksPerThread;

enum { kModeDelta = 0, kModeFirst = 1, kModeSkip = 2 };
enum { kStBadId = 1, kStDupId = 2, kStNoRaw = 4 };

// ------------------------------------------------------------------ 16-bit types

template <typename T> struct Conv;

template <> struct Conv<__half> {
  static __device__ __forceinline__ void unpack(const uint4& v, float (&f)[8]) {
    const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 t = __half22float2(h[i]);
      f[2 * i] = t.x;
      f[2 * i + 1] = t.y;
    }
  }
  static __device__ __forceinline__ uint4 pack(const float (&f)[8]) {
    uint4 v;
    __half2* h = reinterpret_cast<__half2*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2half2_rn(f[2 * i], f[2 * i + 1]);
    return v;
  }
};

template <> struct Conv<__nv_bfloat16> {
  static __device__ __forceinline__ void unpack(const uint4& v, float (&f)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  static __device__ __forceinline__ uint4 pack(const float (&f)[8]) {
    uint4 v;
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    return v;
  }
};

// ------------------------------------------------------------------ quantizer core

// Largest magnitude over the lanes_per_group consecutive lanes that hold one group.
__device__ __forceinline__ float group_max(float s, int lanes_per_group) {
  for (int o = lanes_per_group >> 1; o > 0; o >>= 1) s = fmaxf(s, __shfl_xor_sync(kFullMask, s, o));
  return s;
}

__device__ __forceinline__ float abs_max8(const float (&d)[8]) {
  float s = 0.0f;
#pragma unroll
  for (int j = 0; j < 8; ++j) s = fmaxf(s, fabsf(d[j]));
  return s;
}

// Codes and reconstruction of 8 elements whose group has maximum magnitude s.
//   delta = s * 2^(1-b)  (0 when below FLT_MIN),  k = clamp(floor(d * (1/delta))),
//   q = (k + 1/2) * delta.
// floor and the b-bit field come from one addition rounded toward -inf: for
// |u| <= 128, u + 1.5*2^23 rounded down is 1.5*2^23 + floor(u), whose low mantissa
// bits are the two's-complement code.  Clamping u to [-2^(b-1), 2^(b-1) - 1/2]
// before the floor equals clamping the integer afterwards.
template <int BITS>
__device__ __forceinline__ void quantize8(const float (&d)[8], float s, float& delta,
                                          unsigned long long& codes, float (&q)[8]) {
  constexpr float kTwoPow = 1.0f / (float)(1 << (BITS - 1));
  constexpr float kLo = -(float)(1 << (BITS - 1));
  constexpr float kHi = (float)(1 << (BITS - 1)) - 0.5f;
  constexpr float kMagic = 12582912.0f;
  const float dl = __fmul_rn(s, kTwoPow);
  const bool live = dl >= FLT_MIN;
  delta = live ? dl : 0.0f;
  const float inv = live ? __fdiv_rn(1.0f, dl) : 0.0f;
  codes = 0ull;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    float u = __fmul_rn(d[j], inv);
    u = fminf(fmaxf(u, kLo), kHi);
    const float t = __fadd_rd(u, kMagic);
    const unsigned c = __float_as_uint(t) & ((1u << BITS) - 1u);
    codes |= (unsigned long long)c << (j * BITS);
    const float kf = __fsub_rn(t, kMagic);                 // exact: (float)k
    q[j] = __fmul_rn(__fadd_rn(kf, 0.5f), delta);
  }
}

// q = (k + 1/2) * delta from the b-bit fields.  The field, with its sign bit flipped, is
// placed one bit up in the mantissa of 1.5*2^22 (unit in the last place 1/2) with the lowest
// bit set; subtracting 1.5*2^22 + 2^(b-1) leaves k + 1/2 exactly.
template <int BITS>
__device__ __forceinline__ void dequantize8(unsigned long long codes, float delta, float (&q)[8]) {
  constexpr unsigned kH = 1u << (BITS - 1);
  constexpr unsigned kMask = (1u << BITS) - 1u;
  constexpr float kBias = 6291456.0f + (float)kH;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const unsigned c = (unsigned)(codes >> (j * BITS)) & kMask;
    const float t = __uint_as_float(0x4AC00000u | ((c ^ kH) << 1) | 1u);
    q[j] = __fmul_rn(__fsub_rn(t, kBias), delta);
  }
}

// ------------------------------------------------------------------ bitstream access
// A chunk (8 elements) owns BITS whole bytes at byte offset chunk*BITS of its sample's
// stream; a full warp owns 32*BITS contiguous bytes = 8*BITS words.

template <int BITS>
__device__ __forceinline__ void store_codes(uint8_t* stream, long long chunk, int lane, bool active,
                                            bool warp_words, unsigned long long v) {
  if constexpr (BITS == 8) {
    if (active) *reinterpret_cast<uint2*>(stream + chunk * 8) = make_uint2((unsigned)v, (unsigned)(v >> 32));
  } else if constexpr (BITS == 4) {
    if (active) *reinterpret_cast<uint32_t*>(stream + chunk * 4) = (uint32_t)v;
  } else if constexpr (BITS == 2) {
    if (active) *reinterpret_cast<uint16_t*>(stream + chunk * 2) = (uint16_t)v;
  } else if constexpr (BITS == 1) {
    if (active) stream[chunk] = (uint8_t)v;
  } else {
    constexpr int kBitsPerLane = 8 * BITS;
    constexpr int kWords = 8 * BITS;
    if (warp_words) {   // uniform over the warp: all 32 lanes active, base word-aligned
      uint32_t* wbase = reinterpret_cast<uint32_t*>(stream + (chunk - lane) * BITS);
#pragma unroll
      for (int r = 0; r < (kWords + 31) / 32; ++r) {
        const int w = lane + 32 * r;
        const int bit0 = 32 * w;
        int src = bit0 / kBitsPerLane;
        const int off = bit0 - src * kBitsPerLane;
        src = min(src, 31);
        const int nxt = min(src + 1, 31);
        uint32_t word;
        if constexpr (BITS <= 4) {
          const uint32_t a = __shfl_sync(kFullMask, (uint32_t)v, src);
          const uint32_t b = __shfl_sync(kFullMask, (uint32_t)v, nxt);
          word = a >> off;
          if (off + 32 > kBitsPerLane) word |= b << (kBitsPerLane - off);
        } else {
          const unsigned long long a = __shfl_sync(kFullMask, v, src);
          const unsigned long long b = __shfl_sync(kFullMask, v, nxt);
          word = (uint32_t)(a >> off);
          if (off + 32 > kBitsPerLane) word |= (uint32_t)(b << (kBitsPerLane - off));
        }
        if (w < kWords) wbase[w] = word;
      }
    } else if (active) {
#pragma unroll
      for (int i = 0; i < BITS; ++i) stream[chunk * BITS + i] = (uint8_t)(v >> (8 * i));
    }
  }
}

template <int BITS>
__device__ __forceinline__ unsigned long long load_codes(const uint8_t* stream, long long chunk, int lane,
                                                         bool active, bool warp_words) {
  if constexpr (BITS == 8) {
    if (!active) return 0ull;
    const uint2 t = *reinterpret_cast<const uint2*>(stream + chunk * 8);
    return ((unsigned long long)t.y << 32) | t.x;
  } else if constexpr (BITS == 4) {
    return active ? (unsigned long long)*reinterpret_cast<const uint32_t*>(stream + chunk * 4) : 0ull;
  } else if constexpr (BITS == 2) {
    return active ? (unsigned long long)*reinterpret_cast<const uint16_t*>(stream + chunk * 2) : 0ull;
  } else if constexpr (BITS == 1) {
    return active ? (unsigned long long)stream[chunk] : 0ull;
  } else {
    constexpr int kBitsPerLane = 8 * BITS;
    constexpr int kWords = 8 * BITS;
    constexpr int kNeed = (BITS == 7) ? 3 : 2;      // words a lane's field can straddle
    unsigned long long v = 0ull;
    if (warp_words) {
      const uint32_t* wbase = reinterpret_cast<const uint32_t*>(stream + (chunk - lane) * BITS);
      const uint32_t w0 = (lane < kWords) ? wbase[lane] : 0u;
      uint32_t w1 = 0u;
      if constexpr (kWords > 32) w1 = (lane + 32 < kWords) ? wbase[lane + 32] : 0u;
      const int bit0 = kBitsPerLane * lane;
      const int i0 = bit0 >> 5;
      const int off = bit0 & 31;
      uint32_t x[kNeed];
#pragma unroll
      for (int t = 0; t < kNeed; ++t) {
        const int i = i0 + t;
        const uint32_t lo = __shfl_sync(kFullMask, w0, i & 31);
        uint32_t hi = 0u;
        if constexpr (kWords > 32) hi = __shfl_sync(kFullMask, w1, i & 31);
        x[t] = (i >= 32) ? hi : lo;
      }
      v = (((unsigned long long)x[1] << 32) | x[0]) >> off;
      if constexpr (kNeed == 3) {
        if (off + kBitsPerLane > 64) v |= (unsigned long long)x[2] << (64 - off);
      }
      v &= (1ull << kBitsPerLane) - 1ull;
    } else if (active) {
#pragma unroll
      for (int i = 0; i < BITS; ++i) v |= (unsigned long long)stream[chunk * BITS + i] << (8 * i);
    }
    return v;
  }
}

__device__ __forceinline__ uint4 ld_stream(const void* p) { return __ldcs(reinterpret_cast<const uint4*>(p)); }
__device__ __forceinline__ void st_stream(void* p, const uint4& v) { __stcs(reinterpret_cast<uint4*>(p), v); }

// ------------------------------------------------------------------ sample resolution (Algorithm 1, "if xi not seen before")

// Mode of sample y of the call, computed by the whole CTA (uniform result).
__device__ __forceinline__ int cta_resolve(const State& st, const int32_t* ids, int y, bool need_raw,
                                           bool have_raw, long long& id) {
  id = ids[y];
  const bool bad = id < 0 || id >= st.n_samples;
  int dup = 0;
  for (int p = threadIdx.x; p < y; p += kThreads) dup |= (ids[p] == ids[y]);
  dup = __syncthreads_or(dup);
  if (bad || dup) return kModeSkip;
  if (st.seen[id]) return kModeDelta;
  return (need_raw && !have_raw) ? kModeSkip : kModeFirst;
}

// End of a call.  The seen flags may only change after every CTA has read them, so the CTA
// that arrives last (a counter that wraps back to 0; nobody waits) re-derives each sample's
// mode, marks first visits as seen, writes the optional flags and reports skipped samples.
__device__ __forceinline__ void cta_commit(const State& st, const int32_t* ids, int n_batch, bool need_raw,
                                           bool have_raw, uint8_t* first_flags) {
  __shared__ int s_last;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned total = gridDim.x * gridDim.y;
    s_last = (atomicInc(st.ticket, total - 1u) == total - 1u);
  }
  __syncthreads();
  if (!s_last) return;
  unsigned why = 0;
  for (int y = threadIdx.x; y < n_batch; y += kThreads) {
    const long long id = ids[y];
    int mode;
    if (id < 0 || id >= st.n_samples) {
      mode = kModeSkip;
      why |= kStBadId;
    } else {
      bool dup = false;
      for (int p = 0; p < y; ++p) dup |= (ids[p] == ids[y]);
      if (dup) {
        mode = kModeSkip;
        why |= kStDupId;
      } else if (st.seen[id]) {
        mode = kModeDelta;
      } else if (need_raw && !have_raw) {
        mode = kModeSkip;
        why |= kStNoRaw;
      } else {
        mode = kModeFirst;
      }
    }
    if (first_flags) first_flags[y] = (uint8_t)(mode == kModeFirst);
    if (mode == kModeFirst) st.seen[id] = 1;     // distinct ids: no two threads write one flag
  }
  if (why) atomicOr(st.status, why);
}

// ------------------------------------------------------------------ encode (sender)

template <typename T, int BITS>
__global__ void __launch_bounds__(kThreads) encode_kernel(const State st, const EncodeArgs a) {
  const int y = blockIdx.y;
  const int lane = threadIdx.x & 31;
  long long id;
  const int mode = cta_resolve(st, a.ids, y, false, false, id);

  const T* act = reinterpret_cast<const T*>(a.act) + (long long)y * st.elems;
  uint8_t* stream = a.packed + (long long)y * st.packed_bytes;
  float* scales = a.scales + (long long)y * st.groups;
  const bool words_ok = (st.packed_bytes & 3) == 0;
  const long long c0 = (long long)blockIdx.x * kChunksPerCta + threadIdx.x;

  if (mode == kModeDelta) {
    T* m = reinterpret_cast<T*>(st.m) + id * st.elems;
    uint4 av[kChunksPerThread], mv[kChunksPerThread];
#pragma unroll
    for (int i = 0; i < kChunksPerThread; ++i) {
      const long long c = c0 + i * kThreads;
      av[i] = make_uint4(0, 0, 0, 0);
      mv[i] = make_uint4(0, 0, 0, 0);
      if (c < st.chunks) {
        av[i] = ld_stream(act + c * kChunk);
        mv[i] = ld_stream(m + c * kChunk);
      }
    }
#pragma unroll
    for (int i = 0; i < kChunksPerThread; ++i) {
      const long long c = c0 + i * kThreads;
      const bool active = c < st.chunks;
      float af[8], mf[8], d[8], q[8];
      Conv<T>::unpack(av[i], af);
      Conv<T>::unpack(mv[i], mf);
#pragma unroll
      for (int j = 0; j < 8; ++j) d[j] = __fsub_rn(af[j], mf[j]);
      const float s = group_max(abs_max8(d), st.lanes_per_group);
      float delta;
      unsigned long long codes;
      quantize8<BITS>(d, s, delta, codes, q);
#pragma unroll
      for (int j = 0; j < 8; ++j) mf[j] = __fadd_rn(mf[j], q[j]);
      if (active) {
        st_stream(m + c * kChunk, Conv<T>::pack(mf));
        if ((lane & (st.lanes_per_group - 1)) == 0) scales[c >> st.lg_shift] = delta;
      }
      const bool warp_words = words_ok && (c - lane + 32 <= st.chunks);
      store_codes<BITS>(stream, c, lane, active, warp_words, codes);
    }
  } else {
    // first visit: the activation itself becomes m(xi); skipped sample: nothing is stored.
    // Either way the sample's codes and scales are zero.
    T* m = (mode == kModeFirst) ? reinterpret_cast<T*>(st.m) + id * st.elems : nullptr;
#pragma unroll
    for (int i = 0; i < kChunksPerThread; ++i) {
      const long long c = c0 + i * kThreads;
      const bool active = c < st.chunks;
      if (active) {
        if (m) st_stream(m + c * kChunk, ld_stream(act + c * kChunk));
        if ((lane & (st.lanes_per_group - 1)) == 0) scales[c >> st.lg_shift] = 0.0f;
      }
      const bool warp_words = words_ok && (c - lane + 32 <= st.chunks);
      store_codes<BITS>(stream, c, lane, active, warp_words, 0ull);
    }
  }
  cta_commit(st, a.ids, a.n_batch, false, false, a.first_flags);
}

// ------------------------------------------------------------------ decode (receiver)

template <typename T, int BITS>
__global__ void __launch_bounds__(kThreads) decode_kernel(const State st, const DecodeArgs a) {
  const int y = blockIdx.y;
  const int lane = threadIdx.x & 31;
  long long id;
  const int mode = cta_resolve(st, a.ids, y, true, a.raw != nullptr, id);

  T* out = reinterpret_cast<T*>(a.out) + (long long)y * st.elems;
  const long long c0 = (long long)blockIdx.x * kChunksPerCta + threadIdx.x;

  if (mode == kModeDelta) {
    T* m = reinterpret_cast<T*>(st.m) + id * st.elems;
    const uint8_t* stream = a.packed + (long long)y * st.packed_bytes;
    const float* scales = a.scales + (long long)y * st.groups;
    const bool words_ok = (st.packed_bytes & 3) == 0;
    uint4 mv[kChunksPerThread];
    unsigned long long codes[kChunksPerThread];
    float delta[kChunksPerThread];
#pragma unroll
    for (int i = 0; i < kChunksPerThread; ++i) {
      const long long c = c0 + i * kThreads;
      const bool active = c < st.chunks;
      mv[i] = make_uint4(0, 0, 0, 0);
      delta[i] = 0.0f;
      if (active) {
        mv[i] = ld_stream(m + c * kChunk);
        delta[i] = __ldg(scales + (c >> st.lg_shift));
      }
      const bool warp_words = words_ok && (c - lane + 32 <= st.chunks);
      codes[i] = load_codes<BITS>(stream, c, lane, active, warp_words);
    }
#pragma unroll
    for (int i = 0; i < kChunksPerThread; ++i) {
      const long long c = c0 + i * kThreads;
      if (c < st.chunks) {
        float mf[8], q[8];
        Conv<T>::unpack(mv[i], mf);
        dequantize8<BITS>(codes[i], delta[i], q);
#pragma unroll
        for (int j = 0; j < 8; ++j) mf[j] = __fadd_rn(mf[j], q[j]);
        const uint4 nv = Conv<T>::pack(mf);
        st_stream(m + c * kChunk, nv);
        st_stream(out + c * kChunk, nv);
      }
    }
  } else {
    T* m = (mode == kModeFirst) ? reinterpret_cast<T*>(st.m) + id * st.elems : nullptr;
    const T* raw = (mode == kModeFirst) ? reinterpret_cast<const T*>(a.raw) + (long long)y * st.elems : nullptr;
#pragma unroll
    for (int i = 0; i < kChunksPerThread; ++i) {
      const long long c = c0 + i * kThreads;
      if (c < st.chunks) {
        uint4 v = make_uint4(0, 0, 0, 0);
        if (m) {
          v = ld_stream(raw + c * kChunk);
          st_stream(m + c * kChunk, v);
        }
        st_stream(out + c * kChunk, v);
      }
    }
  }
  cta_commit(st, a.ids, a.n_batch, true, a.raw != nullptr, a.first_flags);
}

// ------------------------------------------------------------------ backward direction: direct quantization

template <typename T, int BITS>
__global__ void __launch_bounds__(kThreads) quant_grad_kernel(const T* __restrict__ grad, long long n_chunks,
                                                              int lanes_per_group, uint8_t* __restrict__ packed,
                                                              float* __restrict__ scales) {
  const int lane = threadIdx.x & 31;
  const int lg_shift = __ffs(lanes_per_group) - 1;
  const long long c0 = (long long)blockIdx.x * kChunksPerCta + threadIdx.x;
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
    const float s = group_max(abs_max8(d), lanes_per_group);
    float delta;
    unsigned long long codes;
    quantize8<BITS>(d, s, delta, codes, q);
    if (active && (lane & (lanes_per_group - 1)) == 0) scales[c >> lg_shift] = delta;
    store_codes<BITS>(packed, c, lane, active, c - lane + 32 <= n_chunks, codes);
  }
}

template <typename T, int BITS>
__global__ void __launch_bounds__(kThreads) dequant_grad_kernel(const uint8_t* __restrict__ packed,
                                                                const float* __restrict__ scales, long long n_chunks,
                                                                int lanes_per_group, T* __restrict__ out) {
  const int lane = threadIdx.x & 31;
  const int lg_shift = __ffs(lanes_per_group) - 1;
  const long long c0 = (long long)blockIdx.x * kChunksPerCta + threadIdx.x;
  unsigned long long codes[kChunksPerThread];
  float delta[kChunksPerThread];
#pragma unroll
  for (int i = 0; i < kChunksPerThread; ++i) {
    const long long c = c0 + i * kThreads;
    const bool active = c < n_chunks;
    delta[i] = active ? __ldg(scales + (c >> lg_shift)) : 0.0f;
    codes[i] = load_codes<BITS>(packed, c, lane, active, c - lane + 32 <= n_chunks);
  }
#pragma unroll
  for (int i = 0; i < kChunksPerThread; ++i) {
    const long long c = c0 + i * kThreads;
    if (c < n_chunks) {
      float q[8];
      dequantize8<BITS>(codes[i], delta[i], q);
      st_stream(out + c * kChunk, Conv<T>::pack(q));
    }
  }
}

// ------------------------------------------------------------------ state digest

__device__ __forceinline__ unsigned long long mix64(unsigned long long index, unsigned long long word) {
  unsigned long long z = index * 0x9E3779B97F4A7C15ull + word;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

__global__ void __launch_bounds__(kThreads) checksum_kernel(const State st, unsigned long long* sum_out) {
  const long long n_vec = st.n_samples * st.chunks;      // 16-byte pieces = 4 words each
  const uint4* mv = reinterpret_cast<const uint4*>(st.m);
  const long long stride = (long long)gridDim.x * kThreads;
  unsigned long long acc = 0ull;
  for (long long v = (long long)blockIdx.x * kThreads + threadIdx.x; v < n_vec; v += stride) {
    const uint4 w = __ldcs(mv + v);
    const unsigned long long i = (unsigned long long)v * 4ull;
    acc += mix64(i, w.x) + mix64(i + 1, w.y) + mix64(i + 2, w.z) + mix64(i + 3, w.w);
  }
  for (long long x = (long long)blockIdx.x * kThreads + threadIdx.x; x < st.n_samples; x += stride)
    acc += mix64((1ull << 40) + (unsigned long long)x, st.seen[x]);
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

// ------------------------------------------------------------------ dispatch

#define AQ_DISPATCH_BITS(T, bits, CALL)                     \
  switch (bits) {                                           \
    case 1: CALL(T, 1); break;                              \
    case 2: CALL(T, 2); break;                              \
    case 3: CALL(T, 3); break;                              \
    case 4: CALL(T, 4); break;                              \
    case 5: CALL(T, 5); break;                              \
    case 6: CALL(T, 6); break;                              \
    case 7: CALL(T, 7); break;                              \
    case 8: CALL(T, 8); break;                              \
    default: return cudaErrorInvalidValue;                  \
  }

#define AQ_DISPATCH(dtype, bits, CALL)                      \
  if ((dtype) == 0) {                                       \
    AQ_DISPATCH_BITS(__half, bits, CALL)                    \
  } else if ((dtype) == 1) {                                \
    AQ_DISPATCH_BITS(__nv_bfloat16, bits, CALL)             \
  } else {                                                  \
    return cudaErrorInvalidValue;                           \
  }

inline unsigned grid_x(long long chunks) { return (unsigned)((chunks + kChunksPerCta - 1) / kChunksPerCta); }

}  // namespace

cudaError_t launch_encode(int dtype, int bits, const State& st, const EncodeArgs& a, cudaStream_t s) {
  if (a.n_batch <= 0) return cudaSuccess;
  const dim3 grid(grid_x(st.chunks), (unsigned)a.n_batch);
#define AQ_CALL(T, B) encode_kernel<T, B><<<grid, kThreads, 0, s>>>(st, a)
  AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
  return cudaGetLastError();
}

cudaError_t launch_decode(int dtype, int bits, const State& st, const DecodeArgs& a, cudaStream_t s) {
  if (a.n_batch <= 0) return cudaSuccess;
  const dim3 grid(grid_x(st.chunks), (unsigned)a.n_batch);
#define AQ_CALL(T, B) decode_kernel<T, B><<<grid, kThreads, 0, s>>>(st, a)
  AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
  return cudaGetLastError();
}

cudaError_t launch_quant_grad(int dtype, int bits, int lanes_per_group, const void* grad, long long n_elems,
                              uint8_t* packed, float* scales, cudaStream_t s) {
  if (n_elems <= 0) return cudaSuccess;
  const long long chunks = n_elems / kChunk;
  const unsigned grid = grid_x(chunks);
#define AQ_CALL(T, B) \
  quant_grad_kernel<T, B><<<grid, kThreads, 0, s>>>(reinterpret_cast<const T*>(grad), chunks, lanes_per_group, packed, scales)
  AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
  return cudaGetLastError();
}

cudaError_t launch_dequant_grad(int dtype, int bits, int lanes_per_group, const uint8_t* packed, const float* scales,
                                long long n_elems, void* out, cudaStream_t s) {
  if (n_elems <= 0) return cudaSuccess;
  const long long chunks = n_elems / kChunk;
  const unsigned grid = grid_x(chunks);
#define AQ_CALL(T, B) \
  dequant_grad_kernel<T, B><<<grid, kThreads, 0, s>>>(packed, scales, chunks, lanes_per_group, reinterpret_cast<T*>(out))
  AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
  return cudaGetLastError();
}

cudaError_t launch_checksum(const State& st, unsigned long long* sum_dev, cudaStream_t s) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const long long n_vec = st.n_samples * st.chunks;
  long long want = (n_vec + kThreads - 1) / kThreads;
  const long long cap = (long long)sms * 8;
  const unsigned grid = (unsigned)(want < 1 ? 1 : (want > cap ? cap : want));
  checksum_kernel<<<grid, kThreads, 0, s>>>(st, sum_dev);
  return cudaGetLastError();
}

}  // namespace aq
