// Device and launch helpers shared by the kernel files of the library: 16-bit conversions, the
// quantizer core, bitstream access, the per-call sample lookup, dispatch over types and bit
// widths, the overlapped launch.  Everything sits in an unnamed namespace, so every file that
// includes this header gets its own copy.
#pragma once

#include "aq_internal.h"

#include <cfloat>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

namespace aq {
namespace {

constexpr unsigned kFullMask = 0xffffffffu;
constexpr int kChunksPerThread = 3;                      // grad kernels: chunks per thread (measured: 2, 3, 4)
constexpr int kChunksPerCta = kThreads * kChunksPerThread;

enum { kModeDelta = 0, kModeFirst = 1, kModeSkip = 2, kModeNothing = 3 };   // kModeNothing: not even zeros can be written
enum { kStBadId = 1, kStDupId = 2, kStNoRaw = 4, kStStaged = 8, kStBadPtr = 16 };

// What the launch layer decides for one encode / decode launch.
struct LaunchPlan {
  int rows_per_cta;        // rows of one sample that a CTA walks; grid = (ceil(rows / rows_per_cta), n_batch)
  unsigned share;          // what a CTA adds to the arrival counter ...
  unsigned first_share;    // ... and what CTA (0,0) adds, so that the grid adds kCallQuantum in all
  // Decode launches are one-dimensional and may taper: CTAs [0, ctas1) walk samples [0, n1), gx1 CTAs of
  // rows_per_cta rows per sample; the CTAs behind them walk the last samples, gx2 CTAs of tail_rows rows each.
  unsigned ctas1, gx1, gx2;
  int n1, tail_rows;
};

// Which sample of the call, and which of its rows, a CTA of a one-dimensional (tapered) grid walks.
struct CtaRows {
  int y;       // sample of the call
  int x;       // the CTA's place among those of the sample
  int rows;    // rows per CTA in this part of the grid
};
__device__ __forceinline__ CtaRows locate_cta(const LaunchPlan& plan) {
  unsigned b = blockIdx.x;
  CtaRows c;
  if (b < plan.ctas1) {
    const unsigned q = b / plan.gx1;
    c.y = (int)q;
    c.x = (int)(b - q * plan.gx1);
    c.rows = plan.rows_per_cta;
  } else {
    b -= plan.ctas1;
    const unsigned q = b / plan.gx2;
    c.y = plan.n1 + (int)q;
    c.x = (int)(b - q * plan.gx2);
    c.rows = plan.tail_rows;
  }
  return c;
}

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
  // d[j] = a_j - m[j]: the mixed-precision subtraction widens a_j exactly and rounds the
  // difference once, the same number as converting first and subtracting in binary32
  static __device__ __forceinline__ void diff(const uint4& a, const float (&m)[8], float (&d)[8]) {
    const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
    for (int i = 0; i < 4; ++i)
      asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tsub.rn.f32.f16 %0, lo, %3;\n\tsub.rn.f32.f16 %1, hi, %4;\n\t}"
          : "=f"(d[2 * i]), "=f"(d[2 * i + 1])
          : "r"(w[i]), "f"(m[2 * i]), "f"(m[2 * i + 1]));
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
  static __device__ __forceinline__ void diff(const uint4& a, const float (&m)[8], float (&d)[8]) {
    const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
    for (int i = 0; i < 4; ++i)
      asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tsub.rn.f32.bf16 %0, lo, %3;\n\tsub.rn.f32.bf16 %1, hi, %4;\n\t}"
          : "=f"(d[2 * i]), "=f"(d[2 * i + 1])
          : "r"(w[i]), "f"(m[2 * i]), "f"(m[2 * i + 1]));
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

// quantize8 for the type at hand.  The wide type (bf16: differences span the whole binary32 exponent
// range) needs the two guards of quantize8 only when a step is extreme; whenever every lane of the
// warp has a step in [2^-125, 2^100] (or a dead group) the narrow form computes the same numbers --
// its reciprocal is normal, so the lower clamp cannot bind, and half the step is exact, so the fused
// reconstruction rounds the same product once -- and the warp takes it.
template <int BITS, bool WIDE, bool STOCH>
__device__ __forceinline__ void quantize8_for(const float (&d)[8], float s, const uint4& noise, float& delta,
                                              unsigned long long& codes, float (&q)[8]) {
  if constexpr (!WIDE || STOCH) {
    quantize8<BITS, WIDE, STOCH>(d, s, noise, delta, codes, q);
  } else {
    const float dl = __fmul_rn(s, 1.0f / (float)(1 << (BITS - 1)));
    const bool tame = !(dl >= FLT_MIN) || (dl >= 0x1p-125f && dl <= 0x1p100f);
    if (__all_sync(kFullMask, tame))
      quantize8<BITS, false, false>(d, s, noise, delta, codes, q);
    else
      quantize8<BITS, true, false>(d, s, noise, delta, codes, q);
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

// Idx: the type chunks are numbered with (int inside a sample, wider in the gradient kernel that
// numbers a whole call): offsets are formed in that type, so 32-bit numbering costs no 64-bit arithmetic.
template <int BITS, typename Idx>
__device__ __forceinline__ void store_codes(uint8_t* stream, Idx chunk, int lane, bool active,
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
    if (warp_words && BITS == 3) {
      // four lanes hold 96 bits = three whole words: lane q of the quad builds word q from its own
      // 24 bits and those of lane q + 1 (one shuffle), the fourth lane stores nothing
      const uint32_t own = (uint32_t)v;
      const uint32_t nxt = __shfl_down_sync(kFullMask, own, 1);
      const int q = lane & 3;
      const uint32_t word = (own >> (8 * q)) | (nxt << (24 - 8 * q));
      if (q < 3) reinterpret_cast<uint32_t*>(stream + (chunk >> 2) * 12)[q] = word;
    } else if (warp_words && BITS == 6) {
      // two lanes hold 96 bits = three whole words: the even lane stores words 0 and 1 (its own 48
      // bits and the low 16 of its neighbour's), the odd lane word 2 (its own high 32)
      const uint32_t lo = (uint32_t)v, hi = (uint32_t)(v >> 32);
      const uint32_t other = __shfl_xor_sync(kFullMask, lo, 1);
      const bool odd = lane & 1;
      uint32_t* w = reinterpret_cast<uint32_t*>(stream + (chunk >> 1) * 12);
      w[odd ? 2 : 0] = odd ? ((lo >> 16) | (hi << 16)) : lo;
      if (!odd) w[1] = hi | (other << 16);
    } else if (warp_words) {   // uniform over the warp: all 32 lanes active, base word-aligned
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

template <int BITS, typename Idx>
__device__ __forceinline__ unsigned long long load_codes(const uint8_t* stream, Idx chunk, int lane,
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
    if (warp_words && BITS == 3) {
      // lane q of a quad owns bits [24q, 24q + 24) of the quad's three words: it reads the two
      // words that hold them (no exchange between lanes) and shifts its field down
      const uint32_t* w = reinterpret_cast<const uint32_t*>(stream + (chunk >> 2) * 12);
      const int q = lane & 3;
      const uint32_t a = __ldg(w + max(q - 1, 0)), b = __ldg(w + min(q, 2));
      v = __funnelshift_r(a, b, (24 * q) & 31) & 0xFFFFFFu;
    } else if (warp_words && BITS == 6) {
      // the even lane of a pair owns bits [0, 48) of the pair's three words, the odd lane bits [48, 96)
      const int odd = lane & 1;
      const uint32_t* w = reinterpret_cast<const uint32_t*>(stream + (chunk >> 1) * 12) + odd;
      const uint32_t a = __ldg(w), b = __ldg(w + 1);
      v = ((((unsigned long long)b << 32) | a) >> (16 * odd)) & 0xFFFFFFFFFFFFull;
    } else if (warp_words) {
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


// ------------------------------------------------------------------ calls and samples (Algorithm 1, the first-visit test)

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
// Asks for `bytes` (a multiple of 16) from the 16-byte aligned address p to be brought into L2:
// one instruction, nothing to wait for, no shared memory.  A CTA's first thread of its second
// warp does this for the rows the CTA is about to walk while the first warp looks the sample up.
__device__ __forceinline__ void prefetch_l2(const void* p, unsigned bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}

__device__ __forceinline__ void overlap_with_neighbours() {
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
// The two halves of the above: between them a CTA may issue hints (prefetches into L2), nothing
// whose value it keeps -- L2 is the point of coherence, so a line fetched early is updated in
// place by the writes of the kernel that is still running.
__device__ __forceinline__ void let_dependents_launch() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void wait_for_predecessor() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Issued by one thread of the CTA ahead of wait_for_predecessor: asks for the CTA's rows of m(xi)
// -- chunks [lo, hi) of the sample at position y of the call -- to be brought into L2.  While
// the CTA is waiting for the previous kernel of the stream to drain, the memory system is not
// busy; when the wait is over the real loads find the rows in L2.  The id and the stamp are read
// past L1 (they may not be final yet) and only steer the hint: an id out of range or a sample
// that looks unseen asks for nothing.
template <typename T>
__device__ __forceinline__ void prefetch_rows_of_m(const State& st, const int32_t* ids, int y, int lo, int hi) {
  if (hi <= lo) return;
  const int32_t id = __ldcg(ids + y);
  if (id < 0 || (long long)id >= st.n_samples) return;
  if (__ldcg(st.seen + id) == 0ull) return;
  const unsigned long long row = st.slot_ids ? (unsigned long long)(unsigned)y : (unsigned long long)(unsigned)id;
  const T* m = reinterpret_cast<const T*>(st.m) + row * (unsigned long long)st.elems;
  prefetch_l2(m + (size_t)lo * kChunk, (unsigned)(hi - lo) * 16u);
}

// What a CTA knows about its sample after open_sample.
struct Sample {
  int mode;
  int32_t id;
  unsigned row;   // the sample's row of st.m: its id, or its position in the call when m(xi) was staged
  const void* buf[4];   // list form of the calls: the sample's own buffers, in the order of BufferLists
};

// The pointer arrays of a list-form call (null entries of `list`: that buffer is not used by the
// call); `needed`: a null pointer in the array is an error, not "absent".
struct BufferLists {
  const void* const* list[4];
  bool needed[4];
};

// Sample y of the call, resolved by warp 0 for the whole CTA (one barrier): its id, whether it
// is in range, whether the id appeared earlier in the call (each lane checks a stride of the
// earlier ids), its "seen" stamp and the call number -- four independent memory operations in
// flight together, the stamp one step behind the id.  Lane 0 of the CTA that owns the sample's
// first row also records the visit: status bit of a skipped sample, first-visit flag, stamp.
// With staged messages (st.slot_ids set) row y of st.m holds m of sample slot_ids[y]; a call
// that brings another id to that position skips the sample.
// List form (lists != null): lane 0 also fetches the sample's buffer pointers; one that is
// missing or not 16-byte aligned makes the sample kModeNothing (nothing read or written for it).
// raw_at: which of the lists holds the raw message of a first visit (-1: none); a null entry
// there means "no raw message for this sample".
// cta_x: the CTA's place among those of its sample, where the grid is not (CTAs of a sample, samples).
__device__ __forceinline__ Sample open_sample(const State& st, const LaunchPlan& plan,
                                              const int32_t* __restrict__ ids, int y, bool need_raw,
                                              bool have_raw, uint8_t* first_flags,
                                              const BufferLists* lists = nullptr, int raw_at = -1,
                                              int cta_x = -1) {
  if (cta_x < 0) cta_x = (int)blockIdx.x;       // two-dimensional grid: x counts the CTAs of a sample
  __shared__ Sample s_sample;
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    unsigned long long call = 0ull;
    if (lane == 0) call = take_call_number(st, plan);
    const void* buf[4] = {nullptr, nullptr, nullptr, nullptr};
    bool bad_ptr = false;
    if (lists && lane == 0) {
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (lists->list[k]) buf[k] = lists->list[k][y];
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (lists->list[k])
          bad_ptr |= (reinterpret_cast<uintptr_t>(buf[k]) & 15u) != 0 || (lists->needed[k] && buf[k] == nullptr);
      if (raw_at >= 0) have_raw = buf[raw_at] != nullptr;
    }
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
      if (bad_ptr) {
        mode = kModeNothing;
        why = kStBadPtr;
      } else if (!in_range) {
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
#pragma unroll
      for (int k = 0; k < 4; ++k) s_sample.buf[k] = buf[k];
      if (cta_x == 0) {                          // once per sample and call
        if (why) atomicOr(st.status, why);
        if (first_flags) first_flags[y] = (uint8_t)(mode == kModeFirst);
        if (mode == kModeFirst) st.seen[id] = call;
      }
    }
  }
  __syncthreads();
  return s_sample;
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

}  // namespace
}  // namespace aq
