// Kernels for previous messages kept at another precision than the activations': 2, 4 or 8 bits
// per element with one step per group, or binary32.

#include "aq_device.cuh"

namespace aq {
namespace {

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
    quantize8_for<MBITS, true, false>(m_new, s2, make_uint4(0, 0, 0, 0), dm2, km2, unused);
    store_codes<MBITS>(m_codes, c, lane, write, false, km2);
    if (write && (lane & (st.lanes_per_group - 1)) == 0) m_scales[c >> st.lg_shift] = dm2;
  }
}

// Delta visit of n rows starting at chunk c0 of one sample: all loads of the rows first, then
// the arithmetic.  FULL: n == kRowsPerIter and every chunk is inside the sample.
template <typename T, int BITS, int MBITS, bool SENDER, bool STOCH, bool FULL>
__device__ __forceinline__ void lowbit_rows(const State& st, const EncodeArgs& ea, uint32_t stream_id, const T* __restrict__ act, const uint8_t* __restrict__ wire_r,
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
        float d[8];
        Conv<T>::diff(av[i], m_deq, d);
        const float s = group_max_any(abs_max8(d), st.lanes_per_group);
        uint4 noise = make_uint4(0, 0, 0, 0);                // the message's rounding; the store's stays deterministic
        if constexpr (STOCH) noise = chunk_noise(ea.seed, ea.epoch, stream_id, (uint32_t)c);
        quantize8_for<BITS, true, STOCH>(d, s, noise, delta[i], codes, q);
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
template <typename T, int BITS, int MBITS, bool SENDER, bool STOCH>
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
  const unsigned long long sid = touch ? (unsigned long long)sample.row : 0ull;     // the sample's row of the store
  uint8_t* m_codes = static_cast<uint8_t*>(st.m) + sid * (unsigned long long)st.m_bytes;
  float* m_scales = (MBITS == 32) ? nullptr : st.m_scales + sid * (unsigned)st.groups;

  int r = blockIdx.x * plan.rows_per_cta;
  const int r_end = min(st.rows, r + plan.rows_per_cta);
  if (mode == kModeDelta) {
    const int whole_end = min(r_end, st.chunks / kThreads);
    for (; r + kRowsPerIter <= whole_end; r += kRowsPerIter)
      lowbit_rows<T, BITS, MBITS, SENDER, STOCH, true>(st, ea, (uint32_t)sample.id, in, wire_r, scale_r, wire_w, scale_w,
                                                       out, m_codes, m_scales, r * kThreads + tid, kRowsPerIter,
                                                       lane, words_ok);
    for (; r < r_end; r += kRowsPerIter)
      lowbit_rows<T, BITS, MBITS, SENDER, STOCH, false>(st, ea, (uint32_t)sample.id, in, wire_r, scale_r, wire_w, scale_w,
                                                        out, m_codes, m_scales, r * kThreads + tid,
                                                        min(kRowsPerIter, r_end - r), lane, words_ok);
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
  LaunchPlan plan = {};
  plan.rows_per_cta = (int)per;
  plan.share = (unsigned)(kCallQuantum / ctas);
  plan.first_share = (unsigned)(kCallQuantum - (unsigned long long)plan.share * (ctas - 1ull));
  return launch_overlapped(kernel, dim3((unsigned)gx, (unsigned)n_batch), s, st, ea, da, plan);
}

#define AQ_DISPATCH_MBITS(T, B, SENDER, STOCH)                                                      \
  switch (st.m_bits) {                                                                              \
    case 2: return launch_lowbit(lowbit_kernel<T, B, 2, SENDER, STOCH>, st, ea, da, n_batch, s);    \
    case 4: return launch_lowbit(lowbit_kernel<T, B, 4, SENDER, STOCH>, st, ea, da, n_batch, s);    \
    case 8: return launch_lowbit(lowbit_kernel<T, B, 8, SENDER, STOCH>, st, ea, da, n_batch, s);    \
    case 32: return launch_lowbit(lowbit_kernel<T, B, 32, SENDER, STOCH>, st, ea, da, n_batch, s);  \
    default: return cudaErrorInvalidValue;                                                          \
  }

}  // namespace

cudaError_t launch_encode_lowbit(int dtype, int bits, const State& st, const EncodeArgs& ea, cudaStream_t s) {
  const DecodeArgs da{};
  const int n_batch = ea.n_batch;
  if (ea.stochastic) {
#define AQ_CALL(T, B) AQ_DISPATCH_MBITS(T, B, true, true)
    AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
  } else {
#define AQ_CALL(T, B) AQ_DISPATCH_MBITS(T, B, true, false)
    AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
  }
  return cudaErrorInvalidValue;
}

cudaError_t launch_decode_lowbit(int dtype, int bits, const State& st, const DecodeArgs& da, cudaStream_t s) {
  const EncodeArgs ea{};
  const int n_batch = da.n_batch;
#define AQ_CALL(T, B) AQ_DISPATCH_MBITS(T, B, false, false)
  AQ_DISPATCH(dtype, bits, AQ_CALL)
#undef AQ_CALL
  return cudaErrorInvalidValue;
}

}  // namespace aq
