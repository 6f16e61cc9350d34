/*
 * UniQL hot-path ORACLE -- test infrastructure, not product code.
 *
 * A plain, slow, scalar fp64 statement of what the compressed-model linear
 * layer computes: a dense contraction over 4-bit group-quantised weights
 * restricted to the retained (sorted, truncated) channels, optionally followed
 * by the rotary embedding on the retained head dimensions.  Only tests, the
 * smoke check and the benchmark's CPU-baseline leg may call it.  It shares no
 * code with the CUDA library.
 *
 * Every function is the definition written out; there is no blocking, fusion
 * or reordering.  OpenMP splits independent output channels across threads,
 * each output is still one sequential fp64 sum in increasing channel order.
 *
 * Pinned by tests/test_oracle_pins.py (integer unpack reference, dense numpy
 * matmul at keep-rate 1, slicing, textbook RoPE, norm / relative-position
 * invariants, closed forms, exact rational brute force).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Number of worker threads the parallel loops use (1 without OpenMP). */
int uniql_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Storage format of the benchmark configuration: two codes per byte, the even
 * input channel in the low nibble.  Row n of W[N,K] occupies K/2 bytes. */
static inline int code_at(const uint8_t* packed, int64_t K, int64_t n, int64_t k) {
  uint8_t byte = packed[n * (K / 2) + k / 2];
  return (k % 2 == 0) ? (byte & 0x0F) : (byte >> 4);
}

/* codes[n*K+k] in 0..15 -> packed[n*K/2 + k/2]. Returns 1 on a bad argument. */
int uniql_oracle_pack_u4(const uint8_t* codes, int64_t N, int64_t K, uint8_t* packed) {
  if (K % 2 != 0) return 1;
  for (int64_t n = 0; n < N; ++n)
    for (int64_t b = 0; b < K / 2; ++b) {
      uint8_t lo = codes[n * K + 2 * b], hi = codes[n * K + 2 * b + 1];
      if (lo > 15 || hi > 15) return 1;
      packed[n * (K / 2) + b] = (uint8_t)(lo | (hi << 4));
    }
  return 0;
}

int uniql_oracle_unpack_u4(const uint8_t* packed, int64_t N, int64_t K, uint8_t* codes) {
  if (K % 2 != 0) return 1;
  for (int64_t n = 0; n < N; ++n)
    for (int64_t k = 0; k < K; ++k) codes[n * K + k] = (uint8_t)code_at(packed, K, n, k);
  return 0;
}

/* Group-wise de-quantisation, w = s * (code - z).  The symmetric quantiser of
 * the paper's Section 3.4 equation (codes clamp(round(W/s), -8, 7)) is the
 * special case code+8 stored, z = 8.  scales / zeros: [N][K/g] as doubles
 * (exact images of the stored fp16 values); the group index is taken on the
 * stored input-channel coordinate. */
int uniql_oracle_dequant(const uint8_t* packed, const double* scales, const double* zeros,
                         int64_t N, int64_t K, int64_t g, double* w) {
  if (g <= 0 || K % g != 0 || K % 2 != 0) return 1;
  int64_t G = K / g;
  for (int64_t n = 0; n < N; ++n)
    for (int64_t k = 0; k < K; ++k) {
      double s = scales[n * G + k / g], z = zeros[n * G + k / g];
      w[n * K + k] = s * ((double)code_at(packed, K, n, k) - z);
    }
  return 0;
}

/* The pruned linear layer (Section 3.4, on-device pruning = keeping the leading
 * sorted channels).  O[0..k_out) and I[0..k_in) list the retained output and
 * input channels in stored coordinates; x is compact, x[m*ldx + t] multiplies
 * stored input channel I[t]; acc[m*k_out + j] is output channel O[j].
 *   acc(m,j) = sum_t x(m,t) * s(O_j, I_t/g) * (code(O_j, I_t) - z(O_j, I_t/g)) + bias(O_j)
 * rows[] (optional, n_rows entries) selects which token rows m are evaluated;
 * NULL means all M rows and acc has M rows, otherwise acc has n_rows rows. */
int uniql_oracle_qlinear(const double* x, int64_t M, int64_t ldx, const uint8_t* packed,
                         const double* scales, const double* zeros, const double* bias,
                         int64_t N, int64_t K, int64_t g, const int32_t* O, int64_t k_out,
                         const int32_t* I, int64_t k_in, const int32_t* rows, int64_t n_rows,
                         double* acc) {
  if (g <= 0 || K % g != 0 || K % 2 != 0) return 1;
  for (int64_t j = 0; j < k_out; ++j)
    if (O[j] < 0 || O[j] >= N) return 2;
  for (int64_t t = 0; t < k_in; ++t)
    if (I[t] < 0 || I[t] >= K) return 2;
  int64_t G = K / g;
  int64_t R = rows ? n_rows : M;
  for (int64_t r = 0; r < R; ++r) {
    int64_t m = rows ? rows[r] : r;
    if (m < 0 || m >= M) return 2;
  }
#pragma omp parallel for schedule(static)
  for (int64_t j = 0; j < k_out; ++j) {
    int64_t n = O[j];
    for (int64_t r = 0; r < R; ++r) {
      int64_t m = rows ? rows[r] : r;
      double sum = 0.0;
      for (int64_t t = 0; t < k_in; ++t) {
        int64_t k = I[t];
        double w = scales[n * G + k / g] * ((double)code_at(packed, K, n, k) - zeros[n * G + k / g]);
        sum += x[m * ldx + t] * w;
      }
      if (bias) sum += bias[n];
      acc[r * k_out + j] = sum;
    }
  }
  return 0;
}

/* Rotary embedding on the retained head dimensions (Section 3.2, MHSA paragraph:
 * RoPE(X) = cos * X + sin * R(X), R([x1,x2]) = [-x2, x1], halves of the head).
 * After symmetric sorting and truncation a head keeps d = head_keep dims laid
 * out [first-half survivors | second-half survivors]; compact pair c consists
 * of columns c and c + d/2 and carries the frequency of its ORIGINAL pair
 * index idx[kv][c], kv = h / (n_heads / n_kv_heads) (Algorithm 6: one index
 * vector per key-value head, shared by its query heads; only half of the
 * symmetric vector is stored).  Angle = pos[m] * theta^(-2 p / head_dim) with
 * the un-pruned head_dim, or pos[m] * inv_freq[p] when a table is given.
 * in / out: [R][n_heads * d] fp64; pos has one entry per row of `in`. */
int uniql_oracle_rope(const double* in, int64_t R, int64_t n_heads, int64_t n_kv_heads,
                      int64_t head_dim, int64_t head_keep, const int32_t* idx,
                      const int32_t* pos, double theta, const double* inv_freq, double* out) {
  if (head_dim % 2 || head_keep % 2 || head_keep > head_dim || n_kv_heads <= 0 ||
      n_heads % n_kv_heads)
    return 1;
  int64_t half = head_keep / 2, rep = n_heads / n_kv_heads;
  for (int64_t i = 0; i < n_kv_heads * half; ++i)
    if (idx[i] < 0 || idx[i] >= head_dim / 2) return 2;
  for (int64_t r = 0; r < R; ++r)
    for (int64_t h = 0; h < n_heads; ++h)
      for (int64_t c = 0; c < half; ++c) {
        int64_t p = idx[(h / rep) * half + c];
        double f = inv_freq ? inv_freq[p] : pow(theta, -2.0 * (double)p / (double)head_dim);
        double phi = (double)pos[r] * f;
        double a = in[r * n_heads * head_keep + h * head_keep + c];
        double b = in[r * n_heads * head_keep + h * head_keep + half + c];
        out[r * n_heads * head_keep + h * head_keep + c] = a * cos(phi) - b * sin(phi);
        out[r * n_heads * head_keep + h * head_keep + half + c] = b * cos(phi) + a * sin(phi);
      }
  return 0;
}

/* ---- gated activation of the MLP block -------------------------------------------------
 * Section 3.2 (MLP paragraph) writes the MLP block as f_MLP(X) = (sigma(X W_g) (.) X W_u) W_d.  Reading taken
 * here: sigma is the SiLU gate of the Llama / Qwen blocks the paper compresses,
 * sigma(t) = t * logistic(t) = t / (1 + exp(-t)), applied element by element.
 * g, u, h: n fp64 values each;  h[i] = sigma(g[i]) * u[i]. */
int uniql_oracle_swiglu(const double* g, const double* u, int64_t n, double* h) {
  if (n < 0) return 1;
  for (int64_t i = 0; i < n; ++i) h[i] = g[i] / (1.0 + exp(-g[i])) * u[i];
  return 0;
}
