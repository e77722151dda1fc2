// CPU checker for the sparse-MoE layer on mixed-bitwidth packed experts.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the layer
// computes, written from the paper (EdgeMoE, arXiv 2308.14352); the tests compare the
// GPU library against it and a benchmark may time it as a CPU baseline.  Nothing in the
// product path may call it, and it shares no code with the GPU library.
//
// What it follows:
//   * Section 3.2 "Choosing the algorithm": channel-wise linear quantisation.  The scale
//     of a channel is its maximum absolute value divided by the range the bitwidth can
//     express; the scale is kept as an extra float16 (or float32) channel; experts are
//     held at INT2 / INT4 / INT8.
//   * Section 3.2: quantised weights are never used as they are; decompression mirrors
//     compression, i.e. w~ = q * s.
//   * Sections 1 and 2.1: each FFN is replaced by N experts, each an independent FFN; a
//     trained router sends every token to its Top-K experts (K = 1 or 2).
//
// Readings taken where the paper is silent (all restated in the design notes):
//   qmax = 2^(b-1) - 1;  IEEE fp32 division and round-half-to-even when quantising, with
//   the *stored* (possibly fp16-rounded) scale;  all-zero group -> scale 0, codes 0;
//   b-bit two's-complement fields, low bits first, K contiguous, rows = output channels;
//   groups are runs of `group` consecutive inputs inside one output channel;
//   ties in Top-K go to the lower expert index;  no biases, no capacity limit;
//   with bf16 activations the hidden vector is rounded once to bf16.
//
// Precision: every sum is accumulated in fp64, in index order.
// Parity pins: see tests/test_oracle_*.py (hand-computed rows, closed forms, library
// routines on special cases, dense brute force).  No function here is unpinned.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

inline int qmax_of(int bits) { return (1 << (bits - 1)) - 1; }

// fp32 -> nearest fp16 (ties to even, subnormals kept) -> fp32
inline float round_to_f16(float v) { return static_cast<float>(static_cast<_Float16>(v)); }

// fp64 -> nearest bf16 (8 significant bits, fp32 exponent range, ties to even), as fp64.
// Done directly on the double so that there is a single rounding.
double round_to_bf16(double v) {
  if (!(std::fabs(v) <= 1.7976931348623157e308)) return v;  // inf / nan unchanged
  if (v == 0.0) return v;
  const double a = std::fabs(v);
  if (a < std::ldexp(1.0, -126)) {
    // subnormal bf16 range: fixed quantum 2^-133
    return std::ldexp(std::nearbyint(std::ldexp(v, 133)), -133);
  }
  int e = 0;
  std::frexp(a, &e);                        // a = m * 2^e, m in [0.5, 1)
  const int q = e - 8;                      // quantum 2^(e-8): 8 significant bits
  double r = std::ldexp(std::nearbyint(std::ldexp(v, -q)), q);
  if (std::fabs(r) >= std::ldexp(1.0, 128)) r = std::copysign(INFINITY, v);
  return r;
}

inline double round_to_f32(double v) { return static_cast<double>(static_cast<float>(v)); }

// read field k of a packed row (two's complement, low bits first)
inline int unpack_field(const uint8_t* row, int k, int bits) {
  const int bitpos = k * bits;
  const int mask = (1 << bits) - 1;
  int f = (row[bitpos >> 3] >> (bitpos & 7)) & mask;
  if (f & (1 << (bits - 1))) f -= (1 << bits);
  return f;
}

// row n of the dequantised matrix: w~[k] = q[n,k] * s[n, k / G]   (Section 3.2, "mirror")
void dequant_row(const uint8_t* packed, const float* scales, int n, int K, int bits, int group,
                 double* out) {
  const int G = group > 0 ? group : K;
  const int ngroups = K / G;
  const uint8_t* row = packed + static_cast<size_t>(n) * (static_cast<size_t>(K) * bits / 8);
  for (int k = 0; k < K; ++k) {
    const double s = static_cast<double>(scales[static_cast<size_t>(n) * ngroups + k / G]);
    out[k] = static_cast<double>(unpack_field(row, k, bits)) * s;
  }
}

inline double silu(double a) { return a / (1.0 + std::exp(-a)); }

}  // namespace

extern "C" {

// ---------------------------------------------------------------------------------------
// Section 3.2: channel-wise linear quantisation of W[N][K] (rows = output channels).
// group == 0: one scale per row; otherwise one scale per `group` consecutive inputs.
// q_out[N][K] receives the integer codes, scales_out[N][K/G] the scales *as stored*
// (after the optional fp16 rounding), widened to fp32.
//
// full_range == 0 (the library's default reading of "the range expressible by the bitwidth"):
//   symmetric codes, -qmax .. qmax with qmax = 2^(b-1) - 1, scale = max-abs / qmax.
// full_range != 0 (the other reading): every code of the two's-complement field is used,
//   -2^(b-1) .. 2^(b-1) - 1, scale = max-abs / 2^(b-1); a weight equal to +max-abs is clamped to
//   the largest positive code.  At 2 bits this gives four levels (-2, -1, 0, 1) instead of three.
// ---------------------------------------------------------------------------------------
int orc_quantize_mode(const float* W, int N, int K, int bits, int group, int scale_is_f16, int full_range,
                      int8_t* q_out, float* scales_out) {
  if (bits != 2 && bits != 4 && bits != 8) return -1;
  const int G = group > 0 ? group : K;
  if (K % G != 0) return -2;
  const int ngroups = K / G;
  const int qmax = qmax_of(bits);
  const int qmin = full_range ? -(1 << (bits - 1)) : -qmax;
  const int range = full_range ? (1 << (bits - 1)) : qmax;  // max-abs is divided by this
  for (int n = 0; n < N; ++n) {
    for (int g = 0; g < ngroups; ++g) {
      const float* w = W + static_cast<size_t>(n) * K + static_cast<size_t>(g) * G;
      float amax = 0.0f;
      for (int k = 0; k < G; ++k) amax = std::max(amax, std::fabs(w[k]));
      float s = amax / static_cast<float>(range);
      if (scale_is_f16) s = round_to_f16(s);
      scales_out[static_cast<size_t>(n) * ngroups + g] = s;
      int8_t* q = q_out + static_cast<size_t>(n) * K + static_cast<size_t>(g) * G;
      for (int k = 0; k < G; ++k) {
        int code = 0;
        if (s != 0.0f) {
          const float r = std::nearbyintf(w[k] / s);  // round half to even
          code = static_cast<int>(std::min(std::max(r, static_cast<float>(qmin)),
                                           static_cast<float>(qmax)));
        }
        q[k] = static_cast<int8_t>(code);
      }
    }
  }
  return 0;
}

int orc_quantize(const float* W, int N, int K, int bits, int group, int scale_is_f16, int8_t* q_out,
                 float* scales_out) {
  return orc_quantize_mode(W, N, K, bits, group, scale_is_f16, 0, q_out, scales_out);
}

// Storage format: element k of row n is a b-bit two's-complement field at bit offset
// (k*b) mod 8 of byte n*(K*b/8) + (k*b)/8.
int orc_pack(const int8_t* q, int N, int K, int bits, uint8_t* packed) {
  if (bits != 2 && bits != 4 && bits != 8) return -1;
  if ((static_cast<size_t>(K) * bits) % 8 != 0) return -2;
  const size_t row_bytes = static_cast<size_t>(K) * bits / 8;
  std::memset(packed, 0, row_bytes * N);
  const int mask = (1 << bits) - 1;
  for (int n = 0; n < N; ++n)
    for (int k = 0; k < K; ++k) {
      const int bitpos = k * bits;
      packed[n * row_bytes + (bitpos >> 3)] |=
          static_cast<uint8_t>((q[static_cast<size_t>(n) * K + k] & mask) << (bitpos & 7));
    }
  return 0;
}

int orc_unpack(const uint8_t* packed, int N, int K, int bits, int8_t* q) {
  if (bits != 2 && bits != 4 && bits != 8) return -1;
  const size_t row_bytes = static_cast<size_t>(K) * bits / 8;
  for (int n = 0; n < N; ++n)
    for (int k = 0; k < K; ++k)
      q[static_cast<size_t>(n) * K + k] = static_cast<int8_t>(unpack_field(packed + n * row_bytes, k, bits));
  return 0;
}

// Section 3.2: decompression, W~[n][k] = q * s, exact in fp64.
int orc_dequantize(const uint8_t* packed, const float* scales, int N, int K, int bits, int group,
                   double* Wt) {
  if (bits != 2 && bits != 4 && bits != 8) return -1;
  for (int n = 0; n < N; ++n) dequant_row(packed, scales, n, K, bits, group, Wt + static_cast<size_t>(n) * K);
  return 0;
}

float orc_round_f16(float v) { return round_to_f16(v); }
double orc_round_bf16(double v) { return round_to_bf16(v); }

// ---------------------------------------------------------------------------------------
// Router and Top-K gating (Sections 1, 2.1).  z = x Wr (+ bias), p = softmax(z) over all
// experts, the K largest logits are selected (ties: lower index), listed in descending
// order.  gate = p[e] (renorm == 0) or p[e] / sum of the selected p (renorm == 1).
// bias: null, or bias[t*bias_stride + e] (bias_stride 0 = one vector for all tokens).
// ---------------------------------------------------------------------------------------
int orc_route(const float* x, int T, int d, const float* Wr, const float* bias, int bias_stride,
              int E, int top_k, int renorm, int32_t* ids, float* gates, float* logits) {
  if (top_k < 1 || top_k > E) return -1;
  std::vector<float> z(E);
  std::vector<double> p(E);
  std::vector<char> taken(E);
  for (int t = 0; t < T; ++t) {
    for (int e = 0; e < E; ++e) {
      double acc = 0.0;
      for (int i = 0; i < d; ++i)
        acc += static_cast<double>(x[static_cast<size_t>(t) * d + i]) * static_cast<double>(Wr[static_cast<size_t>(i) * E + e]);
      if (bias) acc += static_cast<double>(bias[static_cast<size_t>(t) * bias_stride + e]);
      z[e] = static_cast<float>(acc);
      if (logits) logits[static_cast<size_t>(t) * E + e] = z[e];
    }
    double zmax = z[0];
    for (int e = 1; e < E; ++e) zmax = std::max(zmax, static_cast<double>(z[e]));
    double denom = 0.0;
    for (int e = 0; e < E; ++e) { p[e] = std::exp(static_cast<double>(z[e]) - zmax); denom += p[e]; }
    for (int e = 0; e < E; ++e) p[e] /= denom;
    std::fill(taken.begin(), taken.end(), 0);
    double psel = 0.0;
    for (int j = 0; j < top_k; ++j) {
      int best = -1;
      for (int e = 0; e < E; ++e)
        if (!taken[e] && (best < 0 || z[e] > z[best])) best = e;
      taken[best] = 1;
      ids[static_cast<size_t>(t) * top_k + j] = best;
      psel += p[best];
    }
    for (int j = 0; j < top_k; ++j) {
      const double pe = p[ids[static_cast<size_t>(t) * top_k + j]];
      gates[static_cast<size_t>(t) * top_k + j] = static_cast<float>(renorm ? pe / psel : pe);
    }
  }
  return 0;
}

// Token -> expert permutation: stable counting sort of pair indices p = t*k + j by expert.
int orc_permute(const int32_t* ids, int n_pairs, int E, int32_t* counts, int32_t* off, int32_t* perm) {
  for (int e = 0; e < E; ++e) counts[e] = 0;
  for (int p = 0; p < n_pairs; ++p) {
    if (ids[p] < 0 || ids[p] >= E) return -1;
    counts[ids[p]]++;
  }
  off[0] = 0;
  for (int e = 0; e < E; ++e) off[e + 1] = off[e] + counts[e];
  std::vector<int32_t> cursor(off, off + E);
  for (int p = 0; p < n_pairs; ++p) perm[cursor[ids[p]]++] = p;
  return 0;
}

// ---------------------------------------------------------------------------------------
// Expert FFN on the dequantised weights + weighted combine.
//   ReLU experts   (act == 0): h = max(0, x W~in),            o = h W~out
//   SwiGLU experts (act == 1): h = silu(x W~1) * (x W~3),      o = h W~2
//   y[t] = sum_j gate[t,j] * o[pair(t,j)],  j ascending, fp64, rounded to fp32.
// packed / scales: arrays of E*3 pointers, entry e*3+m = matrix m of expert e
// (ReLU: m = 0 W_in, 1 W_out; SwiGLU: m = 0 w1, 1 w3, 2 w2); scales widened to fp32.
// hidden_mode: 0 = h rounded to fp32, 1 = h rounded to bf16.
// h_out (nullable): [T*k][f] hidden vectors per pair, o_out (nullable): [T*k][d] fp64.
// ---------------------------------------------------------------------------------------
int orc_moe_ffn_combine(const float* x, int T, int d, int f, int E, int top_k, int act, int group,
                        int hidden_mode, const int32_t* bits, const uint8_t* const* packed,
                        const float* const* scales, const int32_t* ids, const float* gates,
                        float* y, float* h_out, double* o_out) {
  const int n_pairs = T * top_k;
  std::vector<int32_t> counts(E), off(E + 1), perm(n_pairs);
  if (orc_permute(ids, n_pairs, E, counts.data(), off.data(), perm.data()) != 0) return -1;
  std::vector<double> o(static_cast<size_t>(n_pairs) * d, 0.0);
  const int m_out = (act == 0) ? 1 : 2;
  for (int e = 0; e < E; ++e) {
    const int cnt = counts[e];
    if (cnt == 0) continue;  // only activated experts are evaluated
    const int32_t* pairs = perm.data() + off[e];
    std::vector<double> h(static_cast<size_t>(cnt) * f);
    // first projection(s) and activation
#pragma omp parallel
    {
      std::vector<double> w1(d), w3(act == 1 ? d : 0);
#pragma omp for schedule(static)
      for (int n = 0; n < f; ++n) {
        dequant_row(packed[e * 3 + 0], scales[e * 3 + 0], n, d, bits[e], group, w1.data());
        if (act == 1) dequant_row(packed[e * 3 + 1], scales[e * 3 + 1], n, d, bits[e], group, w3.data());
        for (int c = 0; c < cnt; ++c) {
          const float* xt = x + static_cast<size_t>(pairs[c] / top_k) * d;
          double a = 0.0;
          for (int i = 0; i < d; ++i) a += static_cast<double>(xt[i]) * w1[i];
          double hv;
          if (act == 0) {
            hv = a > 0.0 ? a : 0.0;
          } else {
            double b = 0.0;
            for (int i = 0; i < d; ++i) b += static_cast<double>(xt[i]) * w3[i];
            hv = silu(a) * b;
          }
          hv = hidden_mode == 1 ? round_to_bf16(hv) : round_to_f32(hv);
          h[static_cast<size_t>(c) * f + n] = hv;
        }
      }
    }
    if (h_out)
      for (int c = 0; c < cnt; ++c)
        for (int n = 0; n < f; ++n)
          h_out[static_cast<size_t>(pairs[c]) * f + n] = static_cast<float>(h[static_cast<size_t>(c) * f + n]);
    // second projection
#pragma omp parallel
    {
      std::vector<double> w2(f);
#pragma omp for schedule(static)
      for (int n = 0; n < d; ++n) {
        dequant_row(packed[e * 3 + m_out], scales[e * 3 + m_out], n, f, bits[e], group, w2.data());
        for (int c = 0; c < cnt; ++c) {
          const double* hc = h.data() + static_cast<size_t>(c) * f;
          double a = 0.0;
          for (int j = 0; j < f; ++j) a += hc[j] * w2[j];
          o[static_cast<size_t>(pairs[c]) * d + n] = a;
        }
      }
    }
  }
  for (int t = 0; t < T; ++t)
    for (int n = 0; n < d; ++n) {
      double acc = 0.0;
      for (int j = 0; j < top_k; ++j)
        acc += static_cast<double>(gates[static_cast<size_t>(t) * top_k + j]) * o[(static_cast<size_t>(t) * top_k + j) * d + n];
      y[static_cast<size_t>(t) * d + n] = static_cast<float>(acc);
    }
  if (o_out) std::memcpy(o_out, o.data(), o.size() * sizeof(double));
  return 0;
}

// Spot checks for layers too large to evaluate whole.  orc_hidden_for_pair computes the
// full hidden vector h[f] of one (token, expert) pair, by the same definition as above;
// orc_output_channels then evaluates chosen output channels of that pair.
int orc_hidden_for_pair(const float* xt, int d, int f, int act, int group, int hidden_mode, int bits,
                        const uint8_t* const* packed3, const float* const* scales3, double* h) {
#pragma omp parallel
  {
    std::vector<double> w1(d), w3(act == 1 ? d : 0);
#pragma omp for schedule(static)
    for (int n = 0; n < f; ++n) {
      dequant_row(packed3[0], scales3[0], n, d, bits, group, w1.data());
      if (act == 1) dequant_row(packed3[1], scales3[1], n, d, bits, group, w3.data());
      double a = 0.0;
      for (int i = 0; i < d; ++i) a += static_cast<double>(xt[i]) * w1[i];
      double hv;
      if (act == 0) {
        hv = a > 0.0 ? a : 0.0;
      } else {
        double b = 0.0;
        for (int i = 0; i < d; ++i) b += static_cast<double>(xt[i]) * w3[i];
        hv = silu(a) * b;
      }
      h[n] = hidden_mode == 1 ? round_to_bf16(hv) : round_to_f32(hv);
    }
  }
  return 0;
}

// o[n] = sum_j h[j] * W~out[n][j] for the listed output channels only.
int orc_output_channels(const double* h, int f, int group, int bits, const uint8_t* packed_out,
                        const float* scales_out, const int32_t* channels, int n_channels, double* o) {
  std::vector<double> w2(f);
  for (int c = 0; c < n_channels; ++c) {
    dequant_row(packed_out, scales_out, channels[c], f, bits, group, w2.data());
    double a = 0.0;
    for (int j = 0; j < f; ++j) a += h[j] * w2[j];
    o[c] = a;
  }
  return 0;
}

int orc_num_threads() {
#ifdef _OPENMP
  int n = 1;
#pragma omp parallel
  {
#pragma omp single
    n = omp_get_num_threads();
  }
  return n;
#else
  return 1;
#endif
}

}  // extern "C"
