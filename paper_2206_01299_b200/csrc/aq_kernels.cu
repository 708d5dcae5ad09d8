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

#include "aq_internal.h"

#include <cfloat>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

namespace aq {
namespace {

constexpr unsigned kFullMask = 0xffffffffu;
constexpr int kChunksPerThread = 2;                      // grad kernels: chunks per thread
constexpr int kChunksPerCta = kThreads * kChunksPerThread;

enum { kModeDelta = 0, kModeFirst = 1, kModeSkip = 2 };
enum { kStBadId = 1, kStDupId = 2, kStNoRaw = 4, kStStaged = 8 };

// What the launch layer decides for one encode / decode launch.
struct LaunchPlan {
  int rows_per_cta;        // rows of one sample that a CTA walks; grid = (ceil(rows / rows_per_cta), n_batch)
  unsigned share;          // what a CTA adds to the arrival counter ...
  unsigned first_share;    // ... and what CTA (0,0) adds, so that the grid adds kCallQuantum in all
};

// ------------------------------------------------------------------ 16-bit types

template <typename T> struct Conv;

template <> struct Conv<__half> {
  // |a - m| < 2^17 and every non-zero difference is >= 2^-24: the step Delta and its
  // reciprocal are normal numbers, far from the ends of the binary32 range.
  static constexpr bool kWide = false;
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
  static constexpr bool kWide = true;      // full binary32 exponent range
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

// Largest magnitude over the LPG consecutive lanes that hold one group (LPG = 0: the
// lane count is only known at run time).
template <int LPG>
__device__ __forceinline__ float group_max(float s, int lanes_per_group) {
  if constexpr (LPG == 0) {
    for (int o = lanes_per_group >> 1; o > 0; o >>= 1) s = fmaxf(s, __shfl_xor_sync(kFullMask, s, o));
  } else {
#pragma unroll
    for (int o = LPG >> 1; o > 0; o >>= 1) s = fmaxf(s, __shfl_xor_sync(kFullMask, s, o));
  }
  return s;
}

__device__ __forceinline__ float abs_max8(const float (&d)[8]) {
  float s = 0.0f;
#pragma unroll
  for (int j = 0; j < 8; ++j) s = fmaxf(s, fabsf(d[j]));
  return s;
}

// sum over i < n of x << (i * bits)
__host__ __device__ constexpr uint32_t spread(uint32_t x, int n, int bits) {
  uint32_t r = 0;
  for (int i = 0; i < n; ++i) r += x << (i * bits);
  return r;
}

// n biased words t_i = 0x4B400000 + k_i  ->  the n two's-complement fields k_i mod 2^b laid
// end to end (field i at bit i*b), n*b <= 32.  Horner's rule in wrapping 32-bit arithmetic
// gives sum t_i 2^(ib); adding (h - 0x4B400000) * sum 2^(ib), h = 2^(b-1), turns every
// term into the offset code k_i + h in [0, 2^b), which cannot borrow from its neighbour;
// flipping the top bit of each field turns offset codes into two's complement.
template <int BITS, int N>
__device__ __forceinline__ uint32_t pack_fields(const uint32_t* tb) {
  static_assert(BITS * N <= 32, "fields must fit one word");
  constexpr uint32_t kFlip = spread(1u << (BITS - 1), N, BITS);
  constexpr uint32_t kFix = kFlip - spread(0x4B400000u, N, BITS);
  uint32_t acc = tb[N - 1];
#pragma unroll
  for (int i = N - 2; i >= 0; --i) acc = (acc << BITS) + tb[i];
  return (acc + kFix) ^ kFlip;
}

// Codes and reconstruction of 8 elements whose group has maximum magnitude s.
//   delta = s * 2^(1-b)  (0 when below FLT_MIN),  k = clamp(floor(d * (1/delta))),
//   q = (k + 1/2) * delta.
// * floor and the b-bit field come from one addition rounded toward -inf: for |u| <= 128,
//   u + 1.5*2^23 rounded down is 1.5*2^23 + floor(u), whose low mantissa bits are the
//   two's-complement code.  Clamping u to [-2^(b-1), 2^(b-1) - 1/2] before the floor equals
//   clamping the integer afterwards.
// * WIDE = false (differences of two fp16 values: every non-zero one is at least 2^-24 and the
//   step is far from the ends of the binary32 range) drops two guards that WIDE = true keeps.
// * The lower clamp is only compiled for the wide type: with |d| <= s and a normal
//   reciprocal, |d * RN(1/delta)| < 2^(b-1) * (1 + 2^-24), which rounds to at most 2^(b-1).
// * (k + 1/2) * delta, rounded once, is fma(k, delta, delta/2) whenever delta/2 is exact,
//   i.e. delta >= 2^-125, which always holds for fp16 inputs; the wide type adds 1/2 to k
//   (exact) and multiplies.
// STOCH (the unbiased quantizer that Theorem 3.1 assumes): delta = s / (2^(b-1) - 1/2), so that
// the 2^b levels (k + 1/2) * delta reach from -s to +s, and k = floor(d / delta - 1/2 + r) with
// r uniform in [0,1) from `noise`; both clamps are needed then.
template <int BITS, bool WIDE, bool STOCH>
__device__ __forceinline__ void quantize8(const float (&d)[8], float s, const uint4& noise, float& delta,
                                          unsigned long long& codes, float (&q)[8]) {
  constexpr float kTwoPow = 1.0f / (float)(1 << (BITS - 1));
  constexpr float kTop = (float)(1 << (BITS - 1)) - 0.5f;
  constexpr float kLo = -(float)(1 << (BITS - 1));
  constexpr float kHi = (float)(1 << (BITS - 1)) - 0.5f;
  constexpr float kMagic = 12582912.0f;                      // 1.5 * 2^23 = 0x4B400000
  const float dl = STOCH ? __fdiv_rn(s, kTop) : __fmul_rn(s, kTwoPow);
  const bool live = dl >= FLT_MIN;
  delta = live ? dl : 0.0f;
  const float inv = live ? __frcp_rn(dl) : 0.0f;             // IEEE 1/delta, one rounding
  const float half_delta = __fmul_rn(delta, 0.5f);
  // stochastic rounding: r - 1/2 = (h - 32767.5) * 2^-16 for the element's 16 random bits h
  // (a dead group gets no noise: its codes are 0).  2^22 + h + 1/2 is built in the mantissa.
  const float noise_unit = live ? 1.52587890625e-05f : 0.0f;
  const uint32_t nw[4] = {noise.x, noise.y, noise.z, noise.w};
  uint32_t tb[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    float u = __fmul_rn(d[j], inv);
    if constexpr (STOCH) {
      const uint32_t h = (j & 1) ? (nw[j >> 1] >> 16) : (nw[j >> 1] & 0xFFFFu);
      const float hc = __fsub_rn(__uint_as_float(0x4A800001u | (h << 1)), 4227072.0f);   // h - 32767.5, exact
      u = __fmaf_rn(hc, noise_unit, u);                      // hc * 2^-16 is exact: the same sum, one rounding
    }
    if constexpr (WIDE || STOCH) u = fmaxf(u, kLo);
    u = fminf(u, kHi);
    const float t = __fadd_rd(u, kMagic);
    tb[j] = __float_as_uint(t);
    const float kf = __fsub_rn(t, kMagic);                   // exact: (float)k
    if constexpr (WIDE)
      q[j] = __fmul_rn(__fadd_rn(kf, 0.5f), delta);          // delta / 2 may be inexact below 2^-125
    else
      q[j] = __fmaf_rn(kf, delta, half_delta);
  }
  if constexpr (BITS <= 4) {
    codes = pack_fields<BITS, 8>(tb);
  } else {
    const uint32_t lo = pack_fields<BITS, 4>(tb);
    const uint32_t hi = pack_fields<BITS, 4>(tb + 4);
    codes = (unsigned long long)lo | ((unsigned long long)hi << (4 * BITS));
  }
}

// Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC 2011): the 128 random bits of one
// chunk.  key = the seed's two words; counter = { chunk index in the stream, stream id (sample
// id, or 0xFFFFFFFF for gradients), epoch low word, epoch high word }.  Element j of the chunk
// uses bits [16*(j%2), 16*(j%2)+16) of word j/2.
__device__ __forceinline__ uint4 chunk_noise(unsigned long long seed, unsigned long long epoch, uint32_t stream_id,
                                             uint32_t chunk) {
  uint32_t c0 = chunk, c1 = stream_id, c2 = (uint32_t)epoch, c3 = (uint32_t)(epoch >> 32);
  uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    c0 = hi1 ^ c1 ^ k0;
    c1 = lo1;
    c2 = hi0 ^ c3 ^ k1;
    c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return make_uint4(c0, c1, c2, c3);
}

// q = (k + 1/2) * delta from the b-bit fields.  The field, with its sign bit flipped, is
// placed one bit up in the mantissa of 1.5*2^22 (unit in the last place 1/2) with the lowest
// bit set; subtracting 1.5*2^22 + 2^(b-1) leaves k + 1/2 exactly.
template <int BITS>
__device__ __forceinline__ void dequantize8(unsigned long long codes, float delta, float (&q)[8]) {
  constexpr uint32_t kH = 1u << (BITS - 1);
  constexpr uint32_t kField = ((1u << BITS) - 1u) << 1;
  constexpr uint32_t kBits = 0x4AC00001u | (kH << 1);
  constexpr float kBias = 6291456.0f + (float)kH;
  constexpr int kPerWord = (BITS <= 4) ? 8 : 4;
  const uint32_t w[2] = {(uint32_t)codes, (BITS <= 4) ? 0u : (uint32_t)(codes >> (4 * BITS))};
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const uint32_t x = w[j / kPerWord];
    const int sh = (j % kPerWord) * BITS - 1;
    const uint32_t f = (sh >= 0) ? (x >> sh) : (x << 1);
    const float t = __uint_as_float((f & kField) ^ kBits);
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


// ------------------------------------------------------------------ calls and samples (Algorithm 1, "if xi not seen before")

// Number of the running call, the same in every CTA of the grid, different for every launch on
// the handle.  The handle keeps one 64-bit arrival counter that only grows.  Each CTA adds its
// share of kCallQuantum to it, the shares of one grid adding up to exactly kCallQuantum (the
// first CTA takes the remainder; the launch layer works the shares out), so the counter is a
// multiple of kCallQuantum between launches and every value a CTA gets back from its add lies
// in [c * kCallQuantum, (c+1) * kCallQuantum) for the same c: the number of launches before
// this one.  No CTA has to be the last one, nothing is reset, and a replayed CUDA graph counts
// like any other launch.
__device__ __forceinline__ unsigned long long take_call_number(const State& st, const LaunchPlan& plan) {
  const unsigned mine = (blockIdx.x | blockIdx.y) == 0 ? plan.first_share : plan.share;
  return atomicAdd(st.arrivals, (unsigned long long)mine) / kCallQuantum + kFirstCall;
}

// Programmatic dependent launch: let the next kernel of the stream place its CTAs on the
// multiprocessors while this grid is draining, and do not read anything before the previous
// kernel of the stream has completed and its writes are visible.  (Both are hardware-managed
// and no-ops for neighbours launched the ordinary way.)
__device__ __forceinline__ void overlap_with_neighbours() {
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

// What a CTA knows about its sample after open_sample.
struct Sample {
  int mode;
  int32_t id;
  unsigned row;   // the sample's row of st.m: its id, or its position in the call when m(xi) was staged
};

// Sample y of the call, resolved by warp 0 for the whole CTA (one barrier): its id, whether it
// is in range, whether the id appeared earlier in the call (each lane checks a stride of the
// earlier ids), its "seen" stamp and the call number -- four independent memory operations in
// flight together, the stamp one step behind the id.  Lane 0 of the CTA that owns the sample's
// first row also records the visit: status bit of a skipped sample, first-visit flag, stamp.
// With staged messages (st.slot_ids set) row y of st.m holds m of sample slot_ids[y]; a call
// that brings another id to that position skips the sample.
__device__ __forceinline__ Sample open_sample(const State& st, const LaunchPlan& plan,
                                              const int32_t* __restrict__ ids, int y, bool need_raw,
                                              bool have_raw, uint8_t* first_flags) {
  __shared__ Sample s_sample;
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    unsigned long long call = 0ull;
    if (lane == 0) call = take_call_number(st, plan);
    const int32_t id = ids[y];
    const bool in_range = id >= 0 && (long long)id < st.n_samples;
    int dup = 0;
    for (int q = lane; q < y; q += 32) dup |= (ids[q] == id);
    const unsigned long long stamp = (lane == 0 && in_range) ? __ldcg(st.seen + id) : 0ull;
    const int32_t staged = (lane == 0 && st.slot_ids) ? st.slot_ids[y] : id;
    dup = __any_sync(kFullMask, dup);
    if (lane == 0) {
      int mode;
      unsigned why = 0u;
      if (!in_range) {
        mode = kModeSkip;
        why = kStBadId;
      } else if (dup) {
        mode = kModeSkip;
        why = kStDupId;
      } else if (staged != id) {
        mode = kModeSkip;
        why = kStStaged;
      } else if (stamp != 0ull && stamp != call) {
        mode = kModeDelta;
      } else if (need_raw && !have_raw) {
        mode = kModeSkip;
        why = kStNoRaw;
      } else {
        mode = kModeFirst;
      }
      s_sample.mode = mode;
      s_sample.id = id;
      s_sample.row = st.slot_ids ? (unsigned)y : (unsigned)id;
      if (blockIdx.x == 0) {                     // once per sample and call
        if (why) atomicOr(st.status, why);
        if (first_flags) first_flags[y] = (uint8_t)(mode == kModeFirst);
        if (mode == kModeFirst) st.seen[id] = call;
      }
    }
  }
  __syncthreads();
  return s_sample;
}

// ------------------------------------------------------------------ encode (sender)

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
      {
        float af[8];
        Conv<T>::unpack(av[i], af);
        Conv<T>::unpack(mv[i], mf);
#pragma unroll
        for (int j = 0; j < 8; ++j) d[j] = __fsub_rn(af[j], mf[j]);
      }
      const float s = group_max<LPG>(abs_max8(d), st.lanes_per_group);
      float delta;
      unsigned long long codes;
      uint4 noise = make_uint4(0, 0, 0, 0);
      if constexpr (STOCH) noise = chunk_noise(a.seed, a.epoch, stream_id, (uint32_t)c);
      quantize8<BITS, Conv<T>::kWide, STOCH>(d, s, noise, delta, codes, q);
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
template <int BITS>
constexpr int decode_ctas_per_sm() {
  return (BITS <= 4 || BITS == 8) ? 6 : 4;
}

template <typename T, int BITS, int LPG, bool STOCH>
__global__ void __launch_bounds__(kThreads, STOCH ? 4 : encode_ctas_per_sm<T, BITS>())
    encode_kernel(const State st, const EncodeArgs a, const LaunchPlan plan) {
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int y = blockIdx.y;                                       // sample of the call
  overlap_with_neighbours();
  const Sample sample = open_sample(st, plan, a.ids, y, false, false, a.first_flags);
  const int mode = sample.mode;
  // sizes per sample fit 32 bits (checked at create): 32 x 32 -> 64-bit products
  const unsigned elems = (unsigned)st.elems;
  const T* act = reinterpret_cast<const T*>(a.act) + (unsigned long long)(unsigned)y * elems;
  uint8_t* stream = a.packed + (unsigned long long)(unsigned)y * (unsigned)st.packed_bytes;
  float* scales = a.scales + (unsigned long long)(unsigned)y * (unsigned)st.groups;
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
    for (; r < r_end; ++r) {
      const int c = r * kThreads + tid;
      const bool active = c < st.chunks;
      if (active) {
        if (m) st_stream(m + (size_t)c * kChunk, ld_stream(act + (size_t)c * kChunk));
        if ((lane & (st.lanes_per_group - 1)) == 0) scales[c >> st.lg_shift] = 0.0f;
      }
      const bool warp_words = words_ok && (c - lane + 32 <= st.chunks);
      store_codes<BITS>(stream, c, lane, active, warp_words, 0ull);
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

template <typename T, int BITS>
__global__ void __launch_bounds__(kThreads, decode_ctas_per_sm<BITS>()) decode_kernel(const State st, const DecodeArgs a, const LaunchPlan plan) {
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int y = blockIdx.y;                                       // sample of the call
  overlap_with_neighbours();
  const Sample sample = open_sample(st, plan, a.ids, y, true, a.raw != nullptr, a.first_flags);
  const int mode = sample.mode;
  const unsigned elems = (unsigned)st.elems;
  T* out = reinterpret_cast<T*>(a.out) + (unsigned long long)(unsigned)y * elems;
  int r = blockIdx.x * plan.rows_per_cta;                         // this CTA's rows of the sample: [r, r_end)
  const int r_end = min(st.rows, r + plan.rows_per_cta);

  if (mode == kModeDelta) {
    T* m = reinterpret_cast<T*>(st.m) + (unsigned long long)sample.row * elems;
    const uint8_t* stream = a.packed + (unsigned long long)(unsigned)y * (unsigned)st.packed_bytes;
    const float* scales = a.scales + (unsigned long long)(unsigned)y * (unsigned)st.groups;
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
    const T* raw = first ? reinterpret_cast<const T*>(a.raw) + (unsigned long long)(unsigned)y * elems : nullptr;
    for (; r < r_end; ++r) {
      const int c = r * kThreads + tid;
      if (c < st.chunks) {
        uint4 v = make_uint4(0, 0, 0, 0);
        if (first) {
          v = ld_stream(raw + (size_t)c * kChunk);
          st_stream(m + (size_t)c * kChunk, v);
        }
        st_stream(out + (size_t)c * kChunk, v);
      }
    }
  }
}

// ------------------------------------------------------------------ previous messages kept in MBITS bits per element
//
// The store holds Q(m) instead of m: MBITS-bit codes in the messages' bitstream layout plus one
// fp32 step per group, and every visit works on the dequantized store (the paper's "mz"
// ablation; reading: the same Q as for the messages):
//   m_deq = (km + 1/2) * Delta_m;  sender: Delta_msg = Q_b(a - m_deq);  m_new = m_deq + Delta_msg
//   (fp32);  store <- Q_z(m_new);  the receiver's activation is T(m_new).
// A first visit is the same pass with m_deq = 0 and the activation (the raw message) as the
// update, so both branches end in the same re-quantization.  Differences against an fp32 store
// are not differences of two 16-bit values, hence the guarded (WIDE) quantizer arithmetic.

// Largest magnitude over a group whose lane count is only known at run time (uniform over the grid).
__device__ __forceinline__ float group_max_any(float s, int lanes_per_group) {
  switch (lanes_per_group) {
    case 1: return s;
    case 2: return group_max<2>(s, 2);
    case 4: return group_max<4>(s, 4);
    case 8: return group_max<8>(s, 8);
    case 16: return group_max<16>(s, 16);
    default: return group_max<32>(s, 32);
  }
}

// store <- Q_z(m_new) for one chunk, or m_new itself (MBITS == 32)
template <int MBITS>
__device__ __forceinline__ void lowbit_put(const State& st, uint8_t* m_codes, float* m_scales, int c, int lane,
                                           bool write, const float (&m_new)[8]) {
  if constexpr (MBITS == 32) {
    uint4* m_f32 = reinterpret_cast<uint4*>(m_codes);
    if (write) {
      st_stream(m_f32 + 2 * c, make_uint4(__float_as_uint(m_new[0]), __float_as_uint(m_new[1]), __float_as_uint(m_new[2]),
                                          __float_as_uint(m_new[3])));
      st_stream(m_f32 + 2 * c + 1, make_uint4(__float_as_uint(m_new[4]), __float_as_uint(m_new[5]),
                                              __float_as_uint(m_new[6]), __float_as_uint(m_new[7])));
    }
  } else {
    const float s2 = group_max_any(abs_max8(m_new), st.lanes_per_group);
    unsigned long long km2;
    float dm2, unused[8];
    quantize8<MBITS, true, false>(m_new, s2, make_uint4(0, 0, 0, 0), dm2, km2, unused);
    store_codes<MBITS>(m_codes, c, lane, write, false, km2);
    if (write && (lane & (st.lanes_per_group - 1)) == 0) m_scales[c >> st.lg_shift] = dm2;
  }
}

// Delta visit of n rows starting at chunk c0 of one sample: all loads of the rows first, then
// the arithmetic.  FULL: n == kRowsPerIter and every chunk is inside the sample.
template <typename T, int BITS, int MBITS, bool SENDER, bool FULL>
__device__ __forceinline__ void lowbit_rows(const State& st, const T* __restrict__ act, const uint8_t* __restrict__ wire_r,
                                            const float* __restrict__ scale_r, uint8_t* __restrict__ wire_w,
                                            float* __restrict__ scale_w, T* __restrict__ out, uint8_t* m_codes,
                                            float* m_scales, int c0, int n, int lane, bool words_ok) {
  uint4 av[kRowsPerIter], mlo[kRowsPerIter], mhi[kRowsPerIter];
  unsigned long long km[kRowsPerIter], kw[kRowsPerIter];
  float dm[kRowsPerIter], delta[kRowsPerIter];
  const uint4* m_f32 = reinterpret_cast<const uint4*>(m_codes);
#pragma unroll
  for (int i = 0; i < kRowsPerIter; ++i) {
    const int c = c0 + i * kThreads;
    const bool active = FULL || (i < n && c < st.chunks);
    av[i] = mlo[i] = mhi[i] = make_uint4(0, 0, 0, 0);
    km[i] = kw[i] = 0ull;
    dm[i] = delta[i] = 0.0f;
    if (active) {
      if constexpr (MBITS == 32) {
        mlo[i] = ld_stream(m_f32 + 2 * c);
        mhi[i] = ld_stream(m_f32 + 2 * c + 1);
      } else {
        dm[i] = m_scales[c >> st.lg_shift];
      }
      if (SENDER) av[i] = ld_stream(act + (unsigned)c * (unsigned)kChunk);
      else delta[i] = __ldg(scale_r + (c >> st.lg_shift));
    }
    if (FULL || i < n) {                              // uniform over the CTA
      if constexpr (MBITS != 32) km[i] = load_codes<MBITS>(m_codes, c, lane, active, false);
      if (!SENDER) kw[i] = load_codes<BITS>(wire_r, c, lane, active, words_ok && (FULL || c - lane + 32 <= st.chunks));
    }
  }
#pragma unroll
  for (int i = 0; i < kRowsPerIter; ++i) {
    if (FULL || i < n) {                              // uniform over the CTA
      const int c = c0 + i * kThreads;
      const bool active = FULL || c < st.chunks;
      float m_deq[8], q[8], m_new[8];
      if constexpr (MBITS == 32) {
        const uint32_t w[8] = {mlo[i].x, mlo[i].y, mlo[i].z, mlo[i].w, mhi[i].x, mhi[i].y, mhi[i].z, mhi[i].w};
#pragma unroll
        for (int j = 0; j < 8; ++j) m_deq[j] = __uint_as_float(w[j]);
      } else {
        dequantize8<MBITS>(km[i], dm[i], m_deq);
      }
      unsigned long long codes = 0ull;
      if (SENDER) {
        float af[8], d[8];
        Conv<T>::unpack(av[i], af);
#pragma unroll
        for (int j = 0; j < 8; ++j) d[j] = __fsub_rn(af[j], m_deq[j]);
        const float s = group_max_any(abs_max8(d), st.lanes_per_group);
        quantize8<BITS, true, false>(d, s, make_uint4(0, 0, 0, 0), delta[i], codes, q);
      } else {
        dequantize8<BITS>(kw[i], delta[i], q);
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) m_new[j] = __fadd_rn(m_deq[j], q[j]);
      lowbit_put<MBITS>(st, m_codes, m_scales, c, lane, active, m_new);
      if (SENDER) {
        store_codes<BITS>(wire_w, c, lane, active, words_ok && (FULL || c - lane + 32 <= st.chunks), codes);
        if (active && (lane & (st.lanes_per_group - 1)) == 0) scale_w[c >> st.lg_shift] = delta[i];
      } else if (active) {
        st_stream(out + (unsigned)c * (unsigned)kChunk, Conv<T>::pack(m_new));
      }
    }
  }
}

// CTAs per multiprocessor, measured: the re-quantizing kernels are bound by instruction issue and
// gain from every resident warp; the binary32 store is bound by memory and best at four.
template <typename T, int BITS, int MBITS, bool SENDER>
__global__ void __launch_bounds__(kThreads, MBITS == 32 ? 4 : 6)
    lowbit_kernel(const State st, const EncodeArgs ea, const DecodeArgs da, const LaunchPlan plan) {
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int y = blockIdx.y;
  overlap_with_neighbours();
  const Sample sample = SENDER ? open_sample(st, plan, ea.ids, y, false, false, ea.first_flags)
                               : open_sample(st, plan, da.ids, y, true, da.raw != nullptr, da.first_flags);
  const int mode = sample.mode;
  const unsigned elems = (unsigned)st.elems;
  const unsigned long long row = (unsigned long long)(unsigned)y;
  const T* in = SENDER ? reinterpret_cast<const T*>(ea.act) + row * elems
                       : (mode == kModeFirst ? reinterpret_cast<const T*>(da.raw) + row * elems : nullptr);
  uint8_t* wire_w = SENDER ? ea.packed + row * (unsigned)st.packed_bytes : nullptr;
  float* scale_w = SENDER ? ea.scales + row * (unsigned)st.groups : nullptr;
  const uint8_t* wire_r = SENDER ? nullptr : da.packed + row * (unsigned)st.packed_bytes;
  const float* scale_r = SENDER ? nullptr : da.scales + row * (unsigned)st.groups;
  T* out = SENDER ? nullptr : reinterpret_cast<T*>(da.out) + row * elems;
  const bool words_ok = (st.packed_bytes & 3) == 0;
  const bool touch = mode != kModeSkip;
  const unsigned long long sid = touch ? (unsigned long long)(unsigned)sample.id : 0ull;
  uint8_t* m_codes = static_cast<uint8_t*>(st.m) + sid * (unsigned long long)st.m_bytes;
  float* m_scales = (MBITS == 32) ? nullptr : st.m_scales + sid * (unsigned)st.groups;

  int r = blockIdx.x * plan.rows_per_cta;
  const int r_end = min(st.rows, r + plan.rows_per_cta);
  if (mode == kModeDelta) {
    const int whole_end = min(r_end, st.chunks / kThreads);
    for (; r + kRowsPerIter <= whole_end; r += kRowsPerIter)
      lowbit_rows<T, BITS, MBITS, SENDER, true>(st, in, wire_r, scale_r, wire_w, scale_w, out, m_codes, m_scales,
                                                r * kThreads + tid, kRowsPerIter, lane, words_ok);
    for (; r < r_end; r += kRowsPerIter)
      lowbit_rows<T, BITS, MBITS, SENDER, false>(st, in, wire_r, scale_r, wire_w, scale_w, out, m_codes, m_scales,
                                                 r * kThreads + tid, min(kRowsPerIter, r_end - r), lane, words_ok);
    return;
  }
  // first visit: the activation (the raw message) is the update of an empty store, so this
  // branch ends in the same re-quantization; skipped sample: zero codes, scales and output
  for (; r < r_end; ++r) {
    const int c = r * kThreads + tid;
    const bool active = c < st.chunks;
    float m_new[8];
    uint4 v = make_uint4(0, 0, 0, 0);
    if (mode == kModeFirst && active) v = ld_stream(in + (unsigned)c * (unsigned)kChunk);
    Conv<T>::unpack(v, m_new);
    lowbit_put<MBITS>(st, m_codes, m_scales, c, lane, active && touch, m_new);
    if (SENDER) {
      store_codes<BITS>(wire_w, c, lane, active, words_ok && (c - lane + 32 <= st.chunks), 0ull);
      if (active && (lane & (st.lanes_per_group - 1)) == 0) scale_w[c >> st.lg_shift] = 0.0f;
    } else if (active) {
      st_stream(out + (unsigned)c * (unsigned)kChunk, Conv<T>::pack(m_new));     // zeros for a skipped sample
    }
  }
}

// ------------------------------------------------------------------ backward direction: direct quantization

template <typename T, int BITS, int LPG, bool STOCH>
__global__ void __launch_bounds__(kThreads) quant_grad_kernel(const T* __restrict__ grad, long long n_chunks,
                                                              int lanes_per_group, uint8_t* __restrict__ packed,
                                                              float* __restrict__ scales, unsigned long long seed,
                                                              unsigned long long epoch) {
  const int lane = threadIdx.x & 31;
  const int lg_shift = __ffs(lanes_per_group) - 1;
  const long long c0 = (long long)blockIdx.x * kChunksPerCta + threadIdx.x;
  overlap_with_neighbours();
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
    quantize8<BITS, Conv<T>::kWide, STOCH>(d, s, noise, delta, codes, q);
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
  overlap_with_neighbours();
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
  const long long n_vec = st.n_samples * (long long)st.chunks;      // 16-byte pieces = 4 words each
  const uint4* mv = reinterpret_cast<const uint4*>(st.m);
  const long long stride = (long long)gridDim.x * kThreads;
  unsigned long long acc = 0ull;
  for (long long v = (long long)blockIdx.x * kThreads + threadIdx.x; v < n_vec; v += stride) {
    const uint4 w = __ldcs(mv + v);
    const unsigned long long i = (unsigned long long)v * 4ull;
    acc += mix64(i, w.x) + mix64(i + 1, w.y) + mix64(i + 2, w.z) + mix64(i + 3, w.w);
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

// group sizes 64 and 128 (8 and 16 lanes) get their own instantiation; the rest share one
#define AQ_WITH_LPG(lanes, CALL_LPG)                        \
  switch (lanes) {                                          \
    case 8: CALL_LPG(8); break;                             \
    case 16: CALL_LPG(16); break;                           \
    default: CALL_LPG(0); break;                            \
  }

inline unsigned grid_x(long long chunks) { return (unsigned)((chunks + kChunksPerCta - 1) / kChunksPerCta); }

// Launch with programmatic stream serialisation (see overlap_with_neighbours).
template <typename... KArgs, typename... Args>
cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, cudaStream_t s, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kThreads);
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Several waves of short CTAs: the hardware hands out CTAs in order (x fastest, then the
// sample y), so the CTAs in flight cover one moving window of memory, and a finished CTA is
// replaced at once.  A CTA walks kRowsPerCta rows of one sample when the call is large (its
// per-sample work is then paid once per 8192 elements), fewer when that would leave
// multiprocessors idle.
constexpr int kRowsPerCta = 4;

template <typename K, typename Args>
cudaError_t launch_rows(K kernel, const State& st, const Args& a, cudaStream_t s) {
  if (a.n_batch <= 0) return cudaSuccess;
  const long long total = (long long)a.n_batch * st.rows;
  long long per = st.rows_per_cta;
  if (per <= 0) {
    per = total / ((long long)st.sms * 12);
    per = per < kRowsPerIter ? kRowsPerIter : (per > kRowsPerCta ? kRowsPerCta : per);
  }
  if (per > st.rows) per = st.rows;
  long long gx = (st.rows + per - 1) / per;
  if (gx * a.n_batch > (long long)kCallQuantum) {            // keep every CTA's share of the quantum >= 1
    gx = (long long)kCallQuantum / a.n_batch;
    per = (st.rows + gx - 1) / gx;
    gx = (st.rows + per - 1) / per;
  }
  const unsigned long long ctas = (unsigned long long)gx * (unsigned long long)a.n_batch;
  LaunchPlan plan;
  plan.rows_per_cta = (int)per;
  plan.share = (unsigned)(kCallQuantum / ctas);
  plan.first_share = (unsigned)(kCallQuantum - (unsigned long long)plan.share * (ctas - 1ull));
  return launch_overlapped(kernel, dim3((unsigned)gx, (unsigned)a.n_batch), s, st, a, plan);
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
#define AQ_CALL(T, B) return launch_rows(decode_kernel<T, B>, st, a, s)
  AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
  return cudaErrorInvalidValue;
}

// one launch shape for both directions of the low-precision store
template <typename K>
cudaError_t launch_lowbit(K kernel, const State& st, const EncodeArgs& ea, const DecodeArgs& da, int n_batch,
                          cudaStream_t s) {
  if (n_batch <= 0) return cudaSuccess;
  long long per = st.rows_per_cta > 0 ? st.rows_per_cta : kRowsPerCta;
  if (per > st.rows) per = st.rows;
  long long gx = (st.rows + per - 1) / per;
  if (gx * n_batch > (long long)kCallQuantum) {
    gx = (long long)kCallQuantum / n_batch;
    per = (st.rows + gx - 1) / gx;
    gx = (st.rows + per - 1) / per;
  }
  const unsigned long long ctas = (unsigned long long)gx * (unsigned long long)n_batch;
  LaunchPlan plan;
  plan.rows_per_cta = (int)per;
  plan.share = (unsigned)(kCallQuantum / ctas);
  plan.first_share = (unsigned)(kCallQuantum - (unsigned long long)plan.share * (ctas - 1ull));
  return launch_overlapped(kernel, dim3((unsigned)gx, (unsigned)n_batch), s, st, ea, da, plan);
}

#define AQ_DISPATCH_MBITS(T, B, SENDER)                                                             \
  switch (st.m_bits) {                                                                              \
    case 2: return launch_lowbit(lowbit_kernel<T, B, 2, SENDER>, st, ea, da, n_batch, s);           \
    case 4: return launch_lowbit(lowbit_kernel<T, B, 4, SENDER>, st, ea, da, n_batch, s);           \
    case 8: return launch_lowbit(lowbit_kernel<T, B, 8, SENDER>, st, ea, da, n_batch, s);           \
    case 32: return launch_lowbit(lowbit_kernel<T, B, 32, SENDER>, st, ea, da, n_batch, s);         \
    default: return cudaErrorInvalidValue;                                                          \
  }

cudaError_t launch_encode_lowbit(int dtype, int bits, const State& st, const EncodeArgs& ea, cudaStream_t s) {
  const DecodeArgs da{};
  const int n_batch = ea.n_batch;
#define AQ_CALL(T, B) AQ_DISPATCH_MBITS(T, B, true)
  AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
  return cudaErrorInvalidValue;
}

cudaError_t launch_decode_lowbit(int dtype, int bits, const State& st, const DecodeArgs& da, cudaStream_t s) {
  const EncodeArgs ea{};
  const int n_batch = da.n_batch;
#define AQ_CALL(T, B) AQ_DISPATCH_MBITS(T, B, false)
  AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
  return cudaErrorInvalidValue;
}

cudaError_t launch_quant_grad(int dtype, int bits, int lanes_per_group, const void* grad, long long n_elems,
                              uint8_t* packed, float* scales, bool stochastic, unsigned long long seed,
                              unsigned long long epoch, cudaStream_t s) {
  if (n_elems <= 0) return cudaSuccess;
  const long long chunks = n_elems / kChunk;
  const unsigned grid = grid_x(chunks);
#define AQ_CALL_LPG(L)                                                                                              \
  return stochastic ? launch_overlapped(quant_grad_kernel<T_, B_, L, true>, dim3(grid), s,                          \
                                        reinterpret_cast<const T_*>(grad), chunks, lanes_per_group, packed, scales, \
                                        seed, epoch)                                                                \
                    : launch_overlapped(quant_grad_kernel<T_, B_, L, false>, dim3(grid), s,                         \
                                        reinterpret_cast<const T_*>(grad), chunks, lanes_per_group, packed, scales, \
                                        seed, epoch)
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
  const long long chunks = n_elems / kChunk;
  const unsigned grid = grid_x(chunks);
#define AQ_CALL(T, B) \
  return launch_overlapped(dequant_grad_kernel<T, B>, dim3(grid), s, packed, scales, chunks, lanes_per_group, reinterpret_cast<T*>(out))
  AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
  return cudaGetLastError();
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
