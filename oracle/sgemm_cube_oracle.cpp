// SGEMM-cube CPU oracle.
//
// TEST INFRASTRUCTURE, NOT PRODUCT CODE.  This file is the plain, slow, obviously-correct
// definition that the CUDA path is checked against.  It shares no code with the CUDA path and
// must never be linked, imported or called by it.  Only the tests, the smoke check and the
// benchmark's CPU-baseline leg may use it.
//
// What it computes (paper sections in brackets):
//   * f32 -> f16 conversion, round-to-nearest-even, written at bit level, with gradual
//     underflow and overflow to infinity                       [Sec. 3.3, Eq. fp16_high_low; Sec. 4.1]
//   * the two-word split  hi = fl16(x),  lo = fl16((x - hi) * 2^s)   [Eq. recover_eqn, lines 1-2]
//   * the three-product reconstruction  hi*hi + 2^-s (lo*hi + hi*lo)  with FP32 accumulation
//     in a fixed order, k cut into blocks of kb:
//        termwise     [Eq. termwise]     three streams, combined once at the end
//        elementwise  [Eq. elementwise]  the three block products folded into one accumulator
//        reordered elementwise [Sec. 4.5, last paragraph]  corrections of a block summed first
//   * references: FP64 GEMM, |A||B| in FP64, sequential FP32 GEMM of the unsplit inputs,
//     and the hi*hi product alone (the plain FP16 GEMM contrast)    [Sec. 6.1, 6.2]
//
// Pins (see tests/test_oracle_*.py): the worked example V = 32784 [Sec. 4.2], the residual-class
// probability table [Sec. 4.1], Eq. split_error / split_ineqs / ll_bound / main_bound, an
// exhaustive comparison of the conversion with the host's hardware converter, exact-rational
// brute force on tiny inputs.  No function in this file is "parity unpinned".
//
// Build: g++ -O2 -fopenmp -ffp-contract=off -fno-fast-math -shared -fPIC  (see oracle/build.py).
// -ffp-contract=off and the absence of fast-math keep every FP32 operation an IEEE RN operation.

#include <cstdint>
#include <cstring>
#include <cstdlib>
#include <cmath>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

inline uint32_t f32_bits(float x) { uint32_t w; std::memcpy(&w, &x, 4); return w; }
inline float bits_f32(uint32_t w) { float x; std::memcpy(&x, &w, 4); return x; }

// fl16(x): FP32 bit pattern -> FP16 bit pattern, round-to-nearest, ties-to-even.
// [Sec. 3.3 fixes round-to-nearest-even for the decomposition; Sec. 4.1 for
//  the subnormal range: results below 2^-25 round to zero, the midpoint by ties-to-even.]
uint16_t f16_rn(uint32_t w) {
  const uint16_t sign = (uint16_t)((w >> 16) & 0x8000u);
  const uint32_t mag = w & 0x7FFFFFFFu;
  if (mag > 0x7F800000u) return (uint16_t)(sign | 0x7E00u);  // NaN -> quiet NaN
  if (mag == 0x7F800000u) return (uint16_t)(sign | 0x7C00u); // Inf
  const int E = (int)(mag >> 23);         // biased FP32 exponent
  const uint32_t M = mag & 0x007FFFFFu;   // 23 stored mantissa bits
  if (E == 0) return sign;                // FP32 zero / subnormal: far below 2^-25
  const int e = E - 127;                  // offset exponent E_offset
  if (e > 15) return (uint16_t)(sign | 0x7C00u);  // |x| >= 2^16
  if (e >= -14) {
    // Normal FP16 result: keep 10 mantissa bits, round on the 13 dropped ones.
    uint32_t h = ((uint32_t)(e + 15) << 10) | (M >> 13);
    const uint32_t rem = M & 0x1FFFu;
    if (rem > 0x1000u || (rem == 0x1000u && (h & 1u))) h += 1;  // carry c may bump the exponent;
    return (uint16_t)(sign | h);                                // 0x7BFF + 1 = 0x7C00 = Inf
  }
  // Subnormal FP16 result: q = RNE(|x| * 2^24), an integer in 0..1024 (1024 = smallest normal).
  const uint32_t sig = 0x00800000u | M;   // 24-bit significand, |x| = sig * 2^(e-23)
  const int shift = -e - 1;               // |x| * 2^24 = sig * 2^(e+1) = sig >> shift
  if (shift >= 25) return sign;           // |x| < 2^-25 -> zero
  uint32_t q = sig >> shift;
  const uint32_t rem = sig & ((1u << shift) - 1u);
  const uint32_t half = 1u << (shift - 1);
  if (rem > half || (rem == half && (q & 1u))) q += 1;
  return (uint16_t)(sign | q);
}

// Exact FP16 -> FP32.
uint32_t f16_to_f32(uint16_t h) {
  const uint32_t sign = ((uint32_t)h & 0x8000u) << 16;
  const uint32_t E = (h >> 10) & 0x1Fu;
  const uint32_t M = h & 0x3FFu;
  if (E == 0x1F) return sign | 0x7F800000u | (M << 13);
  if (E != 0) return sign | ((E + 112u) << 23) | (M << 13);
  if (M == 0) return sign;
  // subnormal: value = M * 2^-24; normalise
  int p = 9;
  while (!((M >> p) & 1u)) --p;           // top set bit of M
  const uint32_t frac = (M << (23 - p)) & 0x007FFFFFu;
  return sign | ((uint32_t)(p - 24 + 127) << 23) | frac;
}

// Two-word split [Eq. recover_eqn]: hi = to_half(x); lo = to_half((x - to_single(hi)) * s_f).
// The subtraction and the power-of-two scaling are exact in FP32 [Sec. 3.3, last paragraph],
// so ordinary IEEE float operations are used for them.
inline void split1(float x, int s, uint16_t* hi, uint16_t* lo) {
  const uint16_t h = f16_rn(f32_bits(x));
  const float hf = bits_f32(f16_to_f32(h));
  volatile float r = x - hf;
  volatile float t = r * std::ldexp(1.0f, s);
  *hi = h;
  *lo = f16_rn(f32_bits(t));
}

}  // namespace

extern "C" {

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

uint16_t oracle_f16_rn(uint32_t f32_bits_in) { return f16_rn(f32_bits_in); }
uint32_t oracle_f16_to_f32(uint16_t h) { return f16_to_f32(h); }

void oracle_f16_rn_array(int64_t n, const uint32_t* in, uint16_t* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) out[i] = f16_rn(in[i]);
}

void oracle_f16_to_f32_array(int64_t n, const uint16_t* in, uint32_t* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) out[i] = f16_to_f32(in[i]);
}

// Split a rows x cols row-major FP32 matrix (leading dimension ldx) into FP16 bit patterns
// hi, lo (leading dimension ldh).
void oracle_split(int64_t rows, int64_t cols, const float* X, int64_t ldx,
                  uint16_t* hi, uint16_t* lo, int64_t ldh, int s) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < rows; ++i)
    for (int64_t j = 0; j < cols; ++j)
      split1(X[i * ldx + j], s, &hi[i * ldh + j], &lo[i * ldh + j]);
}

// C = hi_A hi_B + 2^-s (lo_A hi_B + hi_A lo_B), FP32 accumulation.   [Eq. recover_eqn]
//   order 0: termwise [Eq. termwise]; order 1: elementwise [Eq. elementwise]; order 2: the
//   reordered elementwise variant of Sec. 4.5 (last paragraph): per k-block the two corrections
//   are summed first, scaled, added to the block's hi*hi product, and the result is added to the
//   accumulator once:  acc = acc + ((R_A^[g]B^[g] + A^[g]R_B^[g]) / s_f + A^[g]B^[g]).
//   kb: size of a k-block g (one product A^[g] B^[g] is summed from zero over ascending k,
//       every addition an FP32 RN addition; FP16 x FP16 products are exact in FP32 [Sec. 4.4]).
//   Chgemm (optional): the hi*hi stream alone, summed the termwise way.
// A is M x K (lda), B is K x N (ldb), C is M x N (ldc), all row-major.
int oracle_sgemm_cube(int64_t M, int64_t N, int64_t K,
                      const float* A, int64_t lda, const float* B, int64_t ldb,
                      float* C, int64_t ldc, int s, int order, int64_t kb, float* Chgemm,
                      int64_t ldch) {
  if (M < 0 || N < 0 || K < 0 || kb <= 0 || s < 0 || s > 24 || order < 0 || order > 2)
    return 1;
  // Split B once; keep the FP16 words widened (exactly) to FP32 for the loops.
  std::vector<float> Bh((size_t)K * N), Bl((size_t)K * N);
#pragma omp parallel for schedule(static)
  for (int64_t k = 0; k < K; ++k)
    for (int64_t j = 0; j < N; ++j) {
      uint16_t h, l;
      split1(B[k * ldb + j], s, &h, &l);
      Bh[(size_t)k * N + j] = bits_f32(f16_to_f32(h));
      Bl[(size_t)k * N + j] = bits_f32(f16_to_f32(l));
    }
  const float inv_sf = std::ldexp(1.0f, -s);   // 1 / s_f, a power of two: scaling is exact
#pragma omp parallel
  {
    std::vector<float> Phh(N), Plh(N), Phl(N);      // block products P_t^g(i, :)
    std::vector<float> Shh(N), Slh(N), Shl(N);      // termwise streams / Shh = running acc
    std::vector<float> Ah(K), Al(K);
#pragma omp for schedule(dynamic, 1)
    for (int64_t i = 0; i < M; ++i) {
      for (int64_t k = 0; k < K; ++k) {
        uint16_t h, l;
        split1(A[i * lda + k], s, &h, &l);
        Ah[k] = bits_f32(f16_to_f32(h));
        Al[k] = bits_f32(f16_to_f32(l));
      }
      for (int64_t j = 0; j < N; ++j) { Shh[j] = 0.f; Slh[j] = 0.f; Shl[j] = 0.f; }
      for (int64_t k0 = 0; k0 < K; k0 += kb) {
        const int64_t k1 = (k0 + kb < K) ? k0 + kb : K;
        for (int64_t j = 0; j < N; ++j) { Phh[j] = 0.f; Plh[j] = 0.f; Phl[j] = 0.f; }
        for (int64_t k = k0; k < k1; ++k) {
          const float ah = Ah[k], al = Al[k];
          const float* bh = &Bh[(size_t)k * N];
          const float* bl = &Bl[(size_t)k * N];
          for (int64_t j = 0; j < N; ++j) {
            Phh[j] = Phh[j] + ah * bh[j];      // A^[g]   B^[g]
            Plh[j] = Plh[j] + al * bh[j];      // R_A^[g] B^[g]
            Phl[j] = Phl[j] + ah * bl[j];      // A^[g]   R_B^[g]
          }
        }
        if (order == 0) {
          for (int64_t j = 0; j < N; ++j) {
            Shh[j] = Shh[j] + Phh[j];
            Slh[j] = Slh[j] + Plh[j];
            Shl[j] = Shl[j] + Phl[j];
          }
        } else if (order == 1) {
          // ((acc + A^[g]B^[g]) + R_A^[g]B^[g]/s_f) + A^[g]R_B^[g]/s_f
          for (int64_t j = 0; j < N; ++j) {
            float acc = Shh[j];
            acc = acc + Phh[j];
            acc = acc + Plh[j] * inv_sf;
            acc = acc + Phl[j] * inv_sf;
            Shh[j] = acc;
            Slh[j] = Slh[j] + Phh[j];          // hi*hi stream alone, for Chgemm
          }
        } else {
          // acc + ((R_A^[g]B^[g] + A^[g]R_B^[g]) / s_f + A^[g]B^[g])
          for (int64_t j = 0; j < N; ++j) {
            const float cross = Plh[j] + Phl[j];
            const float block = cross * inv_sf + Phh[j];
            Shh[j] = Shh[j] + block;
            Slh[j] = Slh[j] + Phh[j];          // hi*hi stream alone, for Chgemm
          }
        }
      }
      if (order == 0) {
        // The corrections are summed among themselves and meet the dominant stream once.
        for (int64_t j = 0; j < N; ++j) {
          const float cross = Slh[j] + Shl[j];
          C[i * ldc + j] = Shh[j] + cross * inv_sf;
          if (Chgemm) Chgemm[i * ldch + j] = Shh[j];
        }
      } else {
        for (int64_t j = 0; j < N; ++j) {
          C[i * ldc + j] = Shh[j];
          if (Chgemm) Chgemm[i * ldch + j] = Slh[j];
        }
      }
    }
  }
  return 0;
}

// Four-term variant: the full expansion of (hi_A + lo_A/s_f)(hi_B + lo_B/s_f), i.e. Eq.
// recover_eqn with the low-low product that Eq. ll_bound bounds kept instead of dropped:
//   C = hi_A hi_B + 2^-s (lo_A hi_B + hi_A lo_B) + 2^-2s lo_A lo_B.
// Termwise only: each of the four streams is summed in k-blocks of kb as in oracle_sgemm_cube; the
// small terms are combined among themselves, smallest first, and meet the dominant stream once:
//   C = S_hh + ((S_lh + S_hl) 2^-s + S_ll 2^-2s).
int oracle_sgemm_cube_four_term(int64_t M, int64_t N, int64_t K,
                                const float* A, int64_t lda, const float* B, int64_t ldb,
                                float* C, int64_t ldc, int s, int64_t kb) {
  if (M < 0 || N < 0 || K < 0 || kb <= 0 || s < 0 || s > 24) return 1;
  std::vector<float> Bh((size_t)K * N), Bl((size_t)K * N);
#pragma omp parallel for schedule(static)
  for (int64_t k = 0; k < K; ++k)
    for (int64_t j = 0; j < N; ++j) {
      uint16_t h, l;
      split1(B[k * ldb + j], s, &h, &l);
      Bh[(size_t)k * N + j] = bits_f32(f16_to_f32(h));
      Bl[(size_t)k * N + j] = bits_f32(f16_to_f32(l));
    }
  const float inv_sf = std::ldexp(1.0f, -s);
  const float inv_sf2 = std::ldexp(1.0f, -2 * s);
#pragma omp parallel
  {
    std::vector<float> P(4 * (size_t)N), S(4 * (size_t)N);   // hh, lh, hl, ll
    std::vector<float> Ah(K), Al(K);
#pragma omp for schedule(dynamic, 1)
    for (int64_t i = 0; i < M; ++i) {
      for (int64_t k = 0; k < K; ++k) {
        uint16_t h, l;
        split1(A[i * lda + k], s, &h, &l);
        Ah[k] = bits_f32(f16_to_f32(h));
        Al[k] = bits_f32(f16_to_f32(l));
      }
      for (size_t t = 0; t < S.size(); ++t) S[t] = 0.f;
      for (int64_t k0 = 0; k0 < K; k0 += kb) {
        const int64_t k1 = (k0 + kb < K) ? k0 + kb : K;
        for (size_t t = 0; t < P.size(); ++t) P[t] = 0.f;
        for (int64_t k = k0; k < k1; ++k) {
          const float ah = Ah[k], al = Al[k];
          const float* bh = &Bh[(size_t)k * N];
          const float* bl = &Bl[(size_t)k * N];
          for (int64_t j = 0; j < N; ++j) {
            P[j] = P[j] + ah * bh[j];
            P[N + j] = P[N + j] + al * bh[j];
            P[2 * N + j] = P[2 * N + j] + ah * bl[j];
            P[3 * N + j] = P[3 * N + j] + al * bl[j];      // FP16 x FP16: exact in FP32
          }
        }
        for (size_t t = 0; t < S.size(); ++t) S[t] = S[t] + P[t];
      }
      for (int64_t j = 0; j < N; ++j) {
        const float cross = S[N + j] + S[2 * N + j];
        const float small = cross * inv_sf + S[3 * N + j] * inv_sf2;
        C[i * ldc + j] = S[j] + small;
      }
    }
  }
  return 0;
}

// FP64 reference C64 = A B and the matrix |A||B|, both accumulated in double.
void oracle_dgemm_ref(int64_t M, int64_t N, int64_t K,
                      const float* A, int64_t lda, const float* B, int64_t ldb,
                      double* C64, double* ABabs) {
#pragma omp parallel
  {
    std::vector<double> c(N), ab(N);
#pragma omp for schedule(dynamic, 1)
    for (int64_t i = 0; i < M; ++i) {
      for (int64_t j = 0; j < N; ++j) { c[j] = 0.0; ab[j] = 0.0; }
      for (int64_t k = 0; k < K; ++k) {
        const double a = (double)A[i * lda + k];
        const double aa = std::fabs(a);
        const float* b = &B[k * ldb];
        for (int64_t j = 0; j < N; ++j) {
          const double bj = (double)b[j];
          c[j] += a * bj;
          ab[j] += aa * std::fabs(bj);
        }
      }
      for (int64_t j = 0; j < N; ++j) {
        C64[i * N + j] = c[j];
        if (ABabs) ABabs[i * N + j] = ab[j];
      }
    }
  }
}

// Sequential FP32 GEMM of the unsplit inputs: acc = fl(acc + fl(a*b)), k ascending.
void oracle_sgemm_f32(int64_t M, int64_t N, int64_t K,
                      const float* A, int64_t lda, const float* B, int64_t ldb,
                      float* C, int64_t ldc) {
#pragma omp parallel
  {
    std::vector<float> c(N);
#pragma omp for schedule(dynamic, 1)
    for (int64_t i = 0; i < M; ++i) {
      for (int64_t j = 0; j < N; ++j) c[j] = 0.f;
      for (int64_t k = 0; k < K; ++k) {
        const float a = A[i * lda + k];
        const float* b = &B[k * ldb];
        for (int64_t j = 0; j < N; ++j) {
          const float p = a * b[j];
          c[j] = c[j] + p;
        }
      }
      for (int64_t j = 0; j < N; ++j) C[i * ldc + j] = c[j];
    }
  }
}

}  // extern "C"
