// CPU oracle for the AQ-SGD boundary codec.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
// codec computes, written from the paper (Algorithm 1, Algorithm 2 of the
// distributed-view appendix, and the quantizer paragraph of Section 4.1
// "Baselines").  Only the tests, the smoke check and the benchmark's
// cpu_baseline / reference arm may build, load or call it.  It shares no code,
// header, table or constant generator with the CUDA library and neither side
// includes the other.
//
// Arithmetic contract: every floating-point step is ONE IEEE-754 binary32
// operation with round-to-nearest-even (compile with -ffp-contract=off, no
// fast-math).  The 16-bit activation types (IEEE binary16 "fp16", and
// bfloat16 "bf16") are converted by the bit-level routines below, not by a
// compiler extension.
//
// Pins (tests/test_oracle_*.py): conversions against numpy/torch tables,
// hand-derived code vectors, exact-rational brute force of the interval index,
// the error bound Delta/2, sender/receiver buffer identity, first-visit
// identity, zero-delta fixed point, step-change decay, bitstream length, and
// published splitmix64 vectors for the checksum mixer; for the stochastic
// quantizer: Philox4x32-10 known-answer vectors, exact-rational brute force,
// E[Q(d)] = d, level structure.
//
// Parity with the paper authors' own implementation is UNPINNED: the paper
// prints no codes, scales or bit layout; mid-rise reconstruction, the fp32
// step as the transmitted scale and the little-endian two's-complement
// bitstream are readings stated here and in the design notes.

#include <cfloat>
#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

namespace {

// ---------------------------------------------------------------------------
// 16-bit float types, bit level (IEEE 754-2008 binary16; bfloat16 = upper half
// of binary32).
// ---------------------------------------------------------------------------

inline uint32_t f32_bits(float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; }
inline float bits_f32(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }

// binary16 -> binary32, exact for every input.
float half_to_float(uint16_t h) {
  const uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
  const uint32_t expo = (h >> 10) & 0x1Fu;
  const uint32_t frac = h & 0x3FFu;
  if (expo == 0x1Fu) return bits_f32(sign | 0x7F800000u | (frac << 13));  // inf / nan
  if (expo == 0) {
    // subnormal (or zero): value = frac * 2^-24, exactly representable in binary32
    float mag = (float)frac * 5.9604644775390625e-08f;  // 2^-24
    return (sign != 0) ? -mag : mag;
  }
  return bits_f32(sign | ((expo + 112u) << 23) | (frac << 13));
}

// binary32 -> binary16, round to nearest, ties to even; overflow gives inf.
uint16_t float_to_half(float f) {
  const uint32_t x = f32_bits(f);
  const uint16_t sign = (uint16_t)((x >> 16) & 0x8000u);
  const uint32_t mag = x & 0x7FFFFFFFu;
  if (mag >= 0x7F800000u) {                       // inf or nan
    return (mag == 0x7F800000u) ? (uint16_t)(sign | 0x7C00u) : (uint16_t)(sign | 0x7E00u);
  }
  const uint32_t e32 = mag >> 23;                 // biased binary32 exponent
  if (e32 >= 143u) return (uint16_t)(sign | 0x7C00u);   // |f| >= 2^16: beyond every finite half
  if (e32 >= 113u) {                              // result is a normal half (before rounding)
    uint32_t r = ((e32 - 112u) << 10) | ((mag & 0x7FFFFFu) >> 13);
    const uint32_t rem = mag & 0x1FFFu;
    if (rem > 0x1000u || (rem == 0x1000u && (r & 1u))) r += 1;  // carry may reach 0x7C00 = inf
    return (uint16_t)(sign | r);
  }
  // result is a subnormal half (or zero): integer r = RNE(|f| * 2^24)
  if (e32 < 102u) return sign;                    // |f| < 2^-25 rounds to zero (2^-25 itself ties to even = 0)
  const uint32_t m = (mag & 0x7FFFFFu) | 0x800000u;   // 24-bit significand, value = m * 2^(e32-150)
  const uint32_t shift = 126u - e32;              // 14 .. 24
  uint32_t r = m >> shift;
  const uint32_t rem = m & ((1u << shift) - 1u);
  const uint32_t halfway = 1u << (shift - 1u);
  if (rem > halfway || (rem == halfway && (r & 1u))) r += 1;    // may become 0x400 = smallest normal
  return (uint16_t)(sign | r);
}

float bf16_to_float(uint16_t b) { return bits_f32((uint32_t)b << 16); }

// binary32 -> bfloat16, round to nearest, ties to even; overflow gives inf.
uint16_t float_to_bf16(float f) {
  const uint32_t x = f32_bits(f);
  if ((x & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((x >> 16) | 0x0040u);  // quiet nan
  uint32_t r = x >> 16;
  const uint32_t rem = x & 0xFFFFu;
  if (rem > 0x8000u || (rem == 0x8000u && (r & 1u))) r += 1;
  return (uint16_t)r;
}

enum { DT_FP16 = 0, DT_BF16 = 1 };

inline float t_to_float(uint16_t v, int dtype) {
  return dtype == DT_FP16 ? half_to_float(v) : bf16_to_float(v);
}
inline uint16_t float_to_t(float v, int dtype) {
  return dtype == DT_FP16 ? float_to_half(v) : float_to_bf16(v);
}

// ---------------------------------------------------------------------------
// The quantizer Q (Section 4.1, "Baselines": normalise the vector into [-1,1],
// partition [-1,1] uniformly into 2^b intervals, send the b-bit interval
// number).  One "vector" is a group of G consecutive hidden elements.
//
//   s     = max_j |d_j|                          (normaliser: sup-norm)
//   Delta = s * 2^(1-b)                          (width of one interval, un-normalised)
//   k_j   = floor(d_j / Delta), clamped to [-2^(b-1), 2^(b-1)-1]
//           (interval number, counted from the interval whose left edge is 0;
//            d_j = +s lies on the right edge of the last interval and is
//            clamped into it)
//   Q(d)_j = (k_j + 1/2) * Delta                 (interval centre)
//
// Readings fixed here: the quotient is formed as d_j * (1/Delta) with one
// division per group; a group with Delta < FLT_MIN (all-zero or vanishing) has
// Delta = 0 and all codes 0.
// ---------------------------------------------------------------------------

void quantize_group(const float* d, int G, int bits, int32_t* k, float* delta_out) {
  float s = 0.0f;
  for (int j = 0; j < G; ++j) {
    const float a = std::fabs(d[j]);
    if (a > s) s = a;
  }
  const float two_pow = 1.0f / (float)(1 << (bits - 1));   // 2^(1-b), exact
  float delta = s * two_pow;
  if (!(delta >= FLT_MIN)) {
    *delta_out = 0.0f;
    for (int j = 0; j < G; ++j) k[j] = 0;
    return;
  }
  const float inv = 1.0f / delta;
  const float kmin = -(float)(1 << (bits - 1));
  const float kmax = (float)((1 << (bits - 1)) - 1);
  for (int j = 0; j < G; ++j) {
    const float u = d[j] * inv;
    float kf = std::floor(u);
    if (kf < kmin) kf = kmin;
    if (kf > kmax) kf = kmax;
    k[j] = (int32_t)kf;
  }
  *delta_out = delta;
}

inline float reconstruct(int32_t k, float delta) {
  const float centre = (float)k + 0.5f;    // exact
  return centre * delta;
}

// ---------------------------------------------------------------------------
// Unbiased variant of Q (the quantizer that Theorem 3.1 assumes; its footnote
// sketches it as a randomised rounding onto the grid of multiples of 2^-b).  Reading
// fixed here: the 2^b levels are spread evenly over the whole of [-s, s],
//
//   Delta = s / (2^(b-1) - 1/2),   level_k = (k + 1/2) * Delta,  k in [-2^(b-1), 2^(b-1)-1]
//   (level_min = -s, level_max = +s),
//
// and d is rounded to one of its two neighbouring levels with probabilities
// proportional to the distance from the other one:
//
//   k = floor(d / Delta - 1/2 + r),  r uniform in [0,1)    =>  E[level_k] = d  for every |d| <= s.
//
// In fp32, with the random number folded into one addition:
//   delta = s / (2^(b-1) - 0.5f);  inv = 1.0f / delta;
//   t = d * inv + rc,  rc = (h - 32767.5) * 2^-16  for a 16-bit random integer h  (rc = r - 1/2, exact);
//   k = clamp(floor(t)).
// The receiver needs nothing new: it reconstructs (k + 1/2) * Delta from the
// transmitted Delta exactly as before.
//
// Random numbers: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, "Parallel random
// numbers: as easy as 1, 2, 3", SC 2011), a counter-based generator, so that
// any element of any call can be regenerated alone.  One 128-bit output serves
// the 8 elements of a chunk, 16 bits each:
//   key     = { seed low word, seed high word }
//   counter = { chunk index inside the stream, stream id, epoch low word, epoch high word }
//   element j of the chunk uses bits [16*(j%2), 16*(j%2)+16) of output word j/2.
// The stream id is the sample id for activations and 0xFFFFFFFF for gradients.
// ---------------------------------------------------------------------------

void philox4x32_10(const uint32_t counter[4], const uint32_t key[2], uint32_t out[4]) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;      // round multipliers
  const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;      // key schedule (Weyl) increments
  uint32_t c0 = counter[0], c1 = counter[1], c2 = counter[2], c3 = counter[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    const uint64_t p0 = (uint64_t)M0 * c0;
    const uint64_t p1 = (uint64_t)M1 * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    const uint32_t n1 = (uint32_t)p1;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    const uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += W0; k1 += W1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// centred random offsets rc = r - 1/2 of the 8 elements of one chunk
void chunk_offsets(uint64_t seed, uint64_t epoch, uint32_t stream_id, uint32_t chunk, float rc[8]) {
  const uint32_t counter[4] = {chunk, stream_id, (uint32_t)epoch, (uint32_t)(epoch >> 32)};
  const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t w[4];
  philox4x32_10(counter, key, w);
  for (int j = 0; j < 8; ++j) {
    const uint32_t h = (w[j / 2] >> (16 * (j % 2))) & 0xFFFFu;
    rc[j] = ((float)h - 32767.5f) * 1.52587890625e-05f;   // 2^-16; both steps exact
  }
}

// d[0..G) are elements first_elem .. first_elem+G of the stream (first_elem is a multiple of 8)
void quantize_group_stochastic(const float* d, int G, int bits, uint64_t seed, uint64_t epoch,
                               uint32_t stream_id, int64_t first_elem, int32_t* k, float* delta_out) {
  float s = 0.0f;
  for (int j = 0; j < G; ++j) {
    const float a = std::fabs(d[j]);
    if (a > s) s = a;
  }
  const float top = (float)(1 << (bits - 1)) - 0.5f;        // level index of +s, plus 1/2
  const float delta = s / top;
  if (!(delta >= FLT_MIN)) {
    *delta_out = 0.0f;
    for (int j = 0; j < G; ++j) k[j] = 0;
    return;
  }
  const float inv = 1.0f / delta;
  const float kmin = -(float)(1 << (bits - 1));
  const float kmax = (float)((1 << (bits - 1)) - 1);
  float rc[8];
  for (int j = 0; j < G; ++j) {
    if (j % 8 == 0) chunk_offsets(seed, epoch, stream_id, (uint32_t)((first_elem + j) / 8), rc);
    const float u = d[j] * inv;
    const float t = u + rc[j % 8];
    float kf = std::floor(t);
    if (kf < kmin) kf = kmin;
    if (kf > kmax) kf = kmax;
    k[j] = (int32_t)kf;
  }
  *delta_out = delta;
}

// ---------------------------------------------------------------------------
// Bitstream: element j of a stream owns bits [j*b, (j+1)*b); bit t of the
// stream is bit (t mod 8) of byte (t div 8).  The field is the low b bits of
// the two's-complement code.
// ---------------------------------------------------------------------------

void put_code(uint8_t* stream, int64_t j, int bits, int32_t k) {
  const uint32_t field = (uint32_t)k & ((1u << bits) - 1u);
  const int64_t t0 = j * bits;
  for (int i = 0; i < bits; ++i) {
    const int64_t t = t0 + i;
    const uint8_t bit = (uint8_t)((field >> i) & 1u);
    uint8_t& byte = stream[t >> 3];
    byte = (uint8_t)((byte & ~(1u << (t & 7))) | (bit << (t & 7)));
  }
}

int32_t get_code(const uint8_t* stream, int64_t j, int bits) {
  uint32_t field = 0;
  const int64_t t0 = j * bits;
  for (int i = 0; i < bits; ++i) {
    const int64_t t = t0 + i;
    field |= (uint32_t)((stream[t >> 3] >> (t & 7)) & 1u) << i;
  }
  if (field & (1u << (bits - 1))) field |= ~((1u << bits) - 1u);   // sign-extend
  return (int32_t)field;
}

// ---------------------------------------------------------------------------
// State of one side of one boundary: the array m of previous messages, indexed
// by sample and zero-filled as Algorithm 1's initialisation step says,
// and the set of samples seen before.
// ---------------------------------------------------------------------------

struct Side {
  int64_t n_samples;
  int seq, hidden, bits, group, dtype;
  std::vector<uint16_t> m;       // [n_samples][seq][hidden], activation dtype
  std::vector<uint8_t> seen;     // [n_samples]
  uint32_t status;               // sticky: 1 id out of range, 2 duplicate id in a call, 4 first visit at decode with no raw message
  int rounding = 0;              // 0: interval number (deterministic), 1: stochastic, unbiased
  uint64_t seed = 0, epoch = 0;  // stochastic rounding: generator key and the caller's call counter
};

enum { ST_BAD_ID = 1, ST_DUP_ID = 2, ST_NO_RAW = 4 };

// 0 = steady (delta) visit, 1 = first visit, 2 = skipped (bad or repeated id)
int resolve(Side* S, const int32_t* ids, int y) {
  const int64_t id = ids[y];
  if (id < 0 || id >= S->n_samples) { S->status |= ST_BAD_ID; return 2; }
  for (int p = 0; p < y; ++p)
    if (ids[p] == ids[y]) { S->status |= ST_DUP_ID; return 2; }
  return S->seen[id] ? 0 : 1;
}

uint64_t mix64(uint64_t index, uint64_t word) {
  // splitmix64 output function (Steele, Lea, Flood 2014; Vigna's constants)
  uint64_t z = index * 0x9E3779B97F4A7C15ull + word;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// ---------------------------------------------------------------------------
// Previous messages kept at low precision (appendix "Number of Bits for
// Previous Messages": "we perform quantization on m, where mz means that we
// use z bits for previous messages").  The paper gives no formula; reading
// fixed here: m is stored per group of G hidden elements as z-bit codes plus
// one fp32 step, with the same Q as the messages (interval number, centre
// reconstruction, max-abs normaliser), and every visit works on the
// dequantized store:
//
//   m_deq  = (km + 1/2) * Delta_m                 (0 for a group with Delta_m = 0)
//   sender: Delta_msg = Q_b(a - m_deq)            receiver: gets Delta_msg
//   m_new  = m_deq + Delta_msg                    (fp32, one rounding; not rounded to T)
//   store  <- Q_z(m_new);   the receiver's activation is T(m_new)
//   first visit: m_new = a (resp. the raw message), store <- Q_z(m_new), activation = the raw message.
//
// Both sides run the same deterministic steps on the same numbers, so their
// stores stay identical.
// ---------------------------------------------------------------------------

struct SideLow {
  int64_t n_samples;
  int seq, hidden, bits, group, dtype, m_bits;
  std::vector<uint8_t> m_codes;   // [n_samples][seq*hidden*m_bits/8], bitstream layout of the messages
  std::vector<float> m_scales;    // [n_samples][seq*hidden/group], Delta_m of every group
  std::vector<uint8_t> seen;
  uint32_t status;
  int rounding = 0;              // of the messages only (0: interval number, 1: stochastic); the store's own
  uint64_t seed = 0, epoch = 0;  // re-quantization always takes the interval number, so that both sides agree
};

int resolve_low(SideLow* S, const int32_t* ids, int y) {
  const int64_t id = ids[y];
  if (id < 0 || id >= S->n_samples) { S->status |= ST_BAD_ID; return 2; }
  for (int p = 0; p < y; ++p)
    if (ids[p] == ids[y]) { S->status |= ST_DUP_ID; return 2; }
  return S->seen[id] ? 0 : 1;
}

// m_bits == 32: the store is m_new itself, binary32, no steps (the precision of the paper's own
// runs, 6.4 MB per 1024 x 1600 example); the "codes" array then holds the floats.
float load_m(const SideLow* S, const uint8_t* MC, const float* MS, int64_t g, int64_t i) {
  if (S->m_bits == 32) { float v; std::memcpy(&v, MC + 4 * i, 4); return v; }
  return reconstruct(get_code(MC, i, S->m_bits), MS[g]);
}

// store <- Q_z(m_new) for one group
void store_group(SideLow* S, uint8_t* MC, float* MS, int64_t g, const float* m_new, int32_t* km) {
  if (S->m_bits == 32) {
    std::memcpy(MC + 4 * g * S->group, m_new, 4 * (size_t)S->group);
    return;
  }
  float dm;
  quantize_group(m_new, S->group, S->m_bits, km, &dm);
  MS[g] = dm;
  for (int j = 0; j < S->group; ++j) put_code(MC, g * S->group + j, S->m_bits, km[j]);
}

}  // namespace

extern "C" {

// ---- conversions and the bare quantizer, exported so the pins can reach them

float aqo_half_to_float(uint16_t h) { return half_to_float(h); }
uint16_t aqo_float_to_half(float f) { return float_to_half(f); }
float aqo_bf16_to_float(uint16_t h) { return bf16_to_float(h); }
uint16_t aqo_float_to_bf16(float f) { return float_to_bf16(f); }
uint64_t aqo_mix64(uint64_t index, uint64_t word) { return mix64(index, word); }

void aqo_quantize_group(const float* d, int G, int bits, int32_t* k, float* delta) {
  quantize_group(d, G, bits, k, delta);
}
void aqo_philox4x32_10(const uint32_t* counter, const uint32_t* key, uint32_t* out) { philox4x32_10(counter, key, out); }
void aqo_quantize_group_stochastic(const float* d, int G, int bits, uint64_t seed, uint64_t epoch, uint32_t stream_id,
                                   int64_t first_elem, int32_t* k, float* delta) {
  quantize_group_stochastic(d, G, bits, seed, epoch, stream_id, first_elem, k, delta);
}
float aqo_reconstruct(int32_t k, float delta) { return reconstruct(k, delta); }
void aqo_put_code(uint8_t* stream, int64_t j, int bits, int32_t k) { put_code(stream, j, bits, k); }
int32_t aqo_get_code(const uint8_t* stream, int64_t j, int bits) { return get_code(stream, j, bits); }

// ---- one side of one boundary

void* aqo_create(int64_t n_samples, int seq, int hidden, int bits, int group, int dtype) {
  if (n_samples <= 0 || seq <= 0 || hidden <= 0 || bits < 1 || bits > 8 || group <= 0) return nullptr;
  if (hidden % group != 0 || (dtype != DT_FP16 && dtype != DT_BF16)) return nullptr;
  if (((int64_t)seq * hidden * bits) % 8 != 0) return nullptr;
  Side* S = new (std::nothrow) Side();
  if (!S) return nullptr;
  S->n_samples = n_samples; S->seq = seq; S->hidden = hidden;
  S->bits = bits; S->group = group; S->dtype = dtype; S->status = 0;
  S->m.assign((size_t)n_samples * seq * hidden, 0);     // Algorithm 1 starts from an all-zero m
  S->seen.assign((size_t)n_samples, 0);
  return S;
}

void aqo_destroy(void* h) { delete (Side*)h; }

// rounding: 0 = interval number (default), 1 = stochastic; seed and epoch only matter for 1
void aqo_set_rounding(void* h, int rounding, uint64_t seed, uint64_t epoch) {
  Side* S = (Side*)h;
  S->rounding = rounding; S->seed = seed; S->epoch = epoch;
}

const uint16_t* aqo_m(void* h) { return ((Side*)h)->m.data(); }
const uint8_t* aqo_seen(void* h) { return ((Side*)h)->seen.data(); }
uint32_t aqo_status(void* h) { Side* S = (Side*)h; uint32_t s = S->status; S->status = 0; return s; }

// Sender (Algorithm 2, the part run on network a; Algorithm 1, the test whether xi was seen before).
//   act     [n_batch][seq][hidden]  activation a(xi)
//   ids     [n_batch]               sample ids xi
//   packed  [n_batch][seq*hidden*bits/8]   out: bitstream of codes
//   scales  [n_batch][seq][hidden/group]   out: Delta of every group
//   first   [n_batch] or null       out: 1 where the sample was a first visit
// First visit: m(xi) = a(xi) (the full-precision activation is the message),
// codes and scales of that sample are zero.  Otherwise
//   Delta_m = Q(a - m),  m <- m + Delta_m,  codes/scales describe Delta_m.
void aqo_encode(void* h, const uint16_t* act, const int32_t* ids, int n_batch,
                uint8_t* packed, float* scales, uint8_t* first) {
  Side* S = (Side*)h;
  const int64_t E = (int64_t)S->seq * S->hidden;
  const int64_t pbytes = E * S->bits / 8;
  const int64_t ngroups = E / S->group;
  std::vector<float> d(S->group);
  std::vector<int32_t> k(S->group);
  for (int y = 0; y < n_batch; ++y) {
    const uint16_t* a = act + (int64_t)y * E;
    uint8_t* P = packed + (int64_t)y * pbytes;
    float* SC = scales + (int64_t)y * ngroups;
    std::memset(P, 0, (size_t)pbytes);
    for (int64_t g = 0; g < ngroups; ++g) SC[g] = 0.0f;
    const int mode = resolve(S, ids, y);
    if (first) first[y] = (uint8_t)(mode == 1);
    if (mode == 2) continue;
    uint16_t* M = S->m.data() + (int64_t)ids[y] * E;
    if (mode == 1) {
      for (int64_t i = 0; i < E; ++i) M[i] = a[i];
      S->seen[ids[y]] = 1;
      continue;
    }
    for (int64_t g = 0; g < ngroups; ++g) {          // groups never straddle token rows: hidden % group == 0
      const int64_t base = g * S->group;
      for (int j = 0; j < S->group; ++j)
        d[j] = t_to_float(a[base + j], S->dtype) - t_to_float(M[base + j], S->dtype);
      float delta;
      if (S->rounding == 1)
        quantize_group_stochastic(d.data(), S->group, S->bits, S->seed, S->epoch, (uint32_t)ids[y], base, k.data(), &delta);
      else
        quantize_group(d.data(), S->group, S->bits, k.data(), &delta);
      SC[g] = delta;
      for (int j = 0; j < S->group; ++j) {
        put_code(P, base + j, S->bits, k[j]);
        const float qhat = reconstruct(k[j], delta);        // (0 + 1/2) * 0 = 0 for a zero group
        const float sum = t_to_float(M[base + j], S->dtype) + qhat;
        M[base + j] = float_to_t(sum, S->dtype);
      }
    }
  }
}

// Receiver (Algorithm 2, "on network b": m <- m + Delta_m, then m is the
// forward activation).
//   raw  [n_batch][seq][hidden] or null: the uncompressed message of first-visit samples
//   out  [n_batch][seq][hidden]: the activation handed to network b
// A skipped sample (bad id, repeated id, first visit with raw == null) gets an
// all-zero out block and no state change.
void aqo_decode(void* h, const uint8_t* packed, const float* scales, const uint16_t* raw,
                const int32_t* ids, int n_batch, uint16_t* out, uint8_t* first) {
  Side* S = (Side*)h;
  const int64_t E = (int64_t)S->seq * S->hidden;
  const int64_t pbytes = E * S->bits / 8;
  const int64_t ngroups = E / S->group;
  for (int y = 0; y < n_batch; ++y) {
    uint16_t* O = out + (int64_t)y * E;
    int mode = resolve(S, ids, y);
    if (mode == 1 && raw == nullptr) { S->status |= ST_NO_RAW; mode = 2; }
    if (first) first[y] = (uint8_t)(mode == 1);
    if (mode == 2) { for (int64_t i = 0; i < E; ++i) O[i] = 0; continue; }
    uint16_t* M = S->m.data() + (int64_t)ids[y] * E;
    if (mode == 1) {
      const uint16_t* R = raw + (int64_t)y * E;
      for (int64_t i = 0; i < E; ++i) { M[i] = R[i]; O[i] = R[i]; }
      S->seen[ids[y]] = 1;
      continue;
    }
    const uint8_t* P = packed + (int64_t)y * pbytes;
    const float* SC = scales + (int64_t)y * ngroups;
    for (int64_t i = 0; i < E; ++i) {
      const float delta = SC[i / S->group];
      const int32_t k = get_code(P, i, S->bits);
      const float qhat = reconstruct(k, delta);
      const float sum = t_to_float(M[i], S->dtype) + qhat;
      M[i] = float_to_t(sum, S->dtype);
      O[i] = M[i];
    }
  }
}

// Direct quantization of the backward activation-gradient (Algorithm 1, the
// message from machine b back to machine a): same Q, no buffer, no delta.
void aqo_quant_grad(const uint16_t* grad, int64_t n_elems, int bits, int group, int dtype,
                    uint8_t* packed, float* scales) {
  std::vector<float> d(group);
  std::vector<int32_t> k(group);
  std::memset(packed, 0, (size_t)(n_elems * bits / 8));
  for (int64_t g = 0; g < n_elems / group; ++g) {
    const int64_t base = g * group;
    for (int j = 0; j < group; ++j) d[j] = t_to_float(grad[base + j], dtype);
    float delta;
    quantize_group(d.data(), group, bits, k.data(), &delta);
    scales[g] = delta;
    for (int j = 0; j < group; ++j) put_code(packed, base + j, bits, k[j]);
  }
}

// The same with the unbiased stochastic Q (stream id 0xFFFFFFFF; the caller gives every call
// its own epoch value).
void aqo_quant_grad_stochastic(const uint16_t* grad, int64_t n_elems, int bits, int group, int dtype,
                               uint64_t seed, uint64_t epoch, uint8_t* packed, float* scales) {
  std::vector<float> d(group);
  std::vector<int32_t> k(group);
  std::memset(packed, 0, (size_t)(n_elems * bits / 8));
  for (int64_t g = 0; g < n_elems / group; ++g) {
    const int64_t base = g * group;
    for (int j = 0; j < group; ++j) d[j] = t_to_float(grad[base + j], dtype);
    float delta;
    quantize_group_stochastic(d.data(), group, bits, seed, epoch, 0xFFFFFFFFu, base, k.data(), &delta);
    scales[g] = delta;
    for (int j = 0; j < group; ++j) put_code(packed, base + j, bits, k[j]);
  }
}

void aqo_dequant_grad(const uint8_t* packed, const float* scales, int64_t n_elems, int bits,
                      int group, int dtype, uint16_t* out) {
  for (int64_t i = 0; i < n_elems; ++i) {
    const float delta = scales[i / group];
    const float v = reconstruct(get_code(packed, i, bits), delta);
    out[i] = float_to_t(v, dtype);
  }
}

// Order-independent 64-bit digest of the whole state: the m array read as
// little-endian 64-bit words (word i = elements 4i .. 4i+3; a last word that
// the array does not fill is completed with zeros -- the library's shapes,
// multiples of 8 elements per sample, have none), plus the seen set.
// (The digest is a device for comparing two states, not a part of the paper's
// method: any fixed mixer serves as long as both sides of a comparison use
// the same one.)
uint64_t aqo_state_checksum(void* h) {
  Side* S = (Side*)h;
  uint64_t sum = 0;
  const int64_t n = (int64_t)S->m.size(), nwords = (n + 3) / 4;
  for (int64_t i = 0; i < nwords; ++i) {
    uint64_t w = 0;
    for (int e = 0; e < 4 && 4 * i + e < n; ++e) w |= (uint64_t)S->m[4 * i + e] << (16 * e);
    sum += mix64((uint64_t)i, w);
  }
  for (int64_t x = 0; x < S->n_samples; ++x)
    sum += mix64((1ull << 40) + (uint64_t)x, S->seen[x]);
  return sum;
}

// ---- one side of one boundary, previous messages stored in m_bits bits per element

void* aqo_low_create(int64_t n_samples, int seq, int hidden, int bits, int group, int dtype, int m_bits) {
  if (n_samples <= 0 || seq <= 0 || hidden <= 0 || bits < 1 || bits > 8 || group <= 0) return nullptr;
  if (((m_bits < 1 || m_bits > 8) && m_bits != 32) || hidden % group != 0 || (dtype != DT_FP16 && dtype != DT_BF16)) return nullptr;
  const int64_t E = (int64_t)seq * hidden;
  if ((E * bits) % 8 != 0 || (E * m_bits) % 8 != 0) return nullptr;
  SideLow* S = new (std::nothrow) SideLow();
  if (!S) return nullptr;
  S->n_samples = n_samples; S->seq = seq; S->hidden = hidden; S->bits = bits; S->group = group;
  S->dtype = dtype; S->m_bits = m_bits; S->status = 0;
  S->m_codes.assign((size_t)(n_samples * E * m_bits / 8), 0);     // codes 0, steps 0: an all-zero m
  S->m_scales.assign(m_bits == 32 ? 0 : (size_t)(n_samples * E / group), 0.0f);
  S->seen.assign((size_t)n_samples, 0);
  return S;
}
void aqo_low_destroy(void* h) { delete (SideLow*)h; }
void aqo_low_set_rounding(void* h, int rounding, uint64_t seed, uint64_t epoch) {
  SideLow* S = (SideLow*)h;
  S->rounding = rounding; S->seed = seed; S->epoch = epoch;
}
const uint8_t* aqo_low_m_codes(void* h) { return ((SideLow*)h)->m_codes.data(); }
const float* aqo_low_m_scales(void* h) { return ((SideLow*)h)->m_scales.data(); }
const uint8_t* aqo_low_seen(void* h) { return ((SideLow*)h)->seen.data(); }
uint32_t aqo_low_status(void* h) { SideLow* S = (SideLow*)h; uint32_t s = S->status; S->status = 0; return s; }

void aqo_low_encode(void* h, const uint16_t* act, const int32_t* ids, int n_batch, uint8_t* packed, float* scales,
                    uint8_t* first) {
  SideLow* S = (SideLow*)h;
  const int64_t E = (int64_t)S->seq * S->hidden, G = S->group;
  const int64_t pbytes = E * S->bits / 8, ngroups = E / G, mbytes = E * S->m_bits / 8;
  std::vector<float> d(G), m_deq(G), m_new(G);
  std::vector<int32_t> k(G), km(G);
  for (int y = 0; y < n_batch; ++y) {
    const uint16_t* a = act + (int64_t)y * E;
    uint8_t* P = packed + (int64_t)y * pbytes;
    float* SC = scales + (int64_t)y * ngroups;
    std::memset(P, 0, (size_t)pbytes);
    for (int64_t g = 0; g < ngroups; ++g) SC[g] = 0.0f;
    const int mode = resolve_low(S, ids, y);
    if (first) first[y] = (uint8_t)(mode == 1);
    if (mode == 2) continue;
    uint8_t* MC = S->m_codes.data() + (int64_t)ids[y] * mbytes;
    float* MS = S->m_bits == 32 ? nullptr : S->m_scales.data() + (int64_t)ids[y] * ngroups;
    for (int64_t g = 0; g < ngroups; ++g) {
      const int64_t base = g * G;
      if (mode == 1) {
        for (int j = 0; j < G; ++j) m_new[j] = t_to_float(a[base + j], S->dtype);
      } else {
        for (int j = 0; j < G; ++j) {
          m_deq[j] = load_m(S, MC, MS, g, base + j);
          d[j] = t_to_float(a[base + j], S->dtype) - m_deq[j];
        }
        float delta;
        if (S->rounding == 1)
          quantize_group_stochastic(d.data(), (int)G, S->bits, S->seed, S->epoch, (uint32_t)ids[y], base, k.data(), &delta);
        else
          quantize_group(d.data(), (int)G, S->bits, k.data(), &delta);
        SC[g] = delta;
        for (int j = 0; j < G; ++j) {
          put_code(P, base + j, S->bits, k[j]);
          m_new[j] = m_deq[j] + reconstruct(k[j], delta);
        }
      }
      store_group(S, MC, MS, g, m_new.data(), km.data());
    }
    if (mode == 1) S->seen[ids[y]] = 1;
  }
}

void aqo_low_decode(void* h, const uint8_t* packed, const float* scales, const uint16_t* raw, const int32_t* ids,
                    int n_batch, uint16_t* out, uint8_t* first) {
  SideLow* S = (SideLow*)h;
  const int64_t E = (int64_t)S->seq * S->hidden, G = S->group;
  const int64_t pbytes = E * S->bits / 8, ngroups = E / G, mbytes = E * S->m_bits / 8;
  std::vector<float> m_new(G);
  std::vector<int32_t> km(G);
  for (int y = 0; y < n_batch; ++y) {
    uint16_t* O = out + (int64_t)y * E;
    int mode = resolve_low(S, ids, y);
    if (mode == 1 && raw == nullptr) { S->status |= ST_NO_RAW; mode = 2; }
    if (first) first[y] = (uint8_t)(mode == 1);
    if (mode == 2) { for (int64_t i = 0; i < E; ++i) O[i] = 0; continue; }
    uint8_t* MC = S->m_codes.data() + (int64_t)ids[y] * mbytes;
    float* MS = S->m_bits == 32 ? nullptr : S->m_scales.data() + (int64_t)ids[y] * ngroups;
    const uint8_t* P = packed + (int64_t)y * pbytes;
    const float* SC = scales + (int64_t)y * ngroups;
    const uint16_t* R = raw ? raw + (int64_t)y * E : nullptr;
    for (int64_t g = 0; g < ngroups; ++g) {
      const int64_t base = g * G;
      for (int j = 0; j < G; ++j) {
        if (mode == 1) {
          m_new[j] = t_to_float(R[base + j], S->dtype);
          O[base + j] = R[base + j];
        } else {
          const float m_deq = load_m(S, MC, MS, g, base + j);
          m_new[j] = m_deq + reconstruct(get_code(P, base + j, S->bits), SC[g]);
          O[base + j] = float_to_t(m_new[j], S->dtype);
        }
      }
      store_group(S, MC, MS, g, m_new.data(), km.data());
    }
    if (mode == 1) S->seen[ids[y]] = 1;
  }
}

// Digest of a low-precision state: the code bytes read as little-endian 32-bit words, then the
// steps' bit patterns (word index continuing), then the seen set as for the 16-bit state.
uint64_t aqo_low_state_checksum(void* h) {
  SideLow* S = (SideLow*)h;
  uint64_t sum = 0;
  const int64_t ncw = (int64_t)S->m_codes.size() / 4;
  for (int64_t i = 0; i < ncw; ++i) {
    uint32_t w;
    std::memcpy(&w, S->m_codes.data() + 4 * i, 4);
    sum += mix64((uint64_t)i, w);
  }
  for (int64_t i = 0; i < (int64_t)S->m_scales.size(); ++i)
    sum += mix64((uint64_t)(ncw + i), f32_bits(S->m_scales[i]));
  for (int64_t x = 0; x < S->n_samples; ++x)
    sum += mix64((1ull << 40) + (uint64_t)x, S->seen[x]);
  return sum;
}

}  // extern "C"
