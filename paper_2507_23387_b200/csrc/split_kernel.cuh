// Operand split kernel (paper Eq. recover_eqn, first two lines; Sec. 3.3; Sec. 4.2):
//   hi = fl16(x),  lo = fl16((x - hi) * 2^s),  both conversions round-to-nearest-even.
// HBM-bound: 4 bytes read and 2 + 2 bytes written per element.  The vector path moves 32 bytes of
// FP32 in (two 16-byte loads) and one 16-byte store to each of hi and lo per thread and item.
#pragma once

#include <cstdint>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

namespace sgc {

// One element.  x - hi is exact in FP32 and so is the power-of-two scaling (Sec. 3.3), so the
// only roundings are the two conversions.  FP16 subnormals are produced, never flushed.
__device__ __forceinline__ void split_one(float x, float scale, uint16_t& hi, uint16_t& lo) {
  const __half h = __float2half_rn(x);
  const float r = __fsub_rn(x, __half2float(h));
  const __half l = __float2half_rn(__fmul_rn(r, scale));
  hi = __half_as_ushort(h);
  lo = __half_as_ushort(l);
}

// Two elements packed: hi and lo words as f16x2 (element 0 in the low half).
__device__ __forceinline__ void split_two(float x0, float x1, float scale, uint32_t& hi2,
                                          uint32_t& lo2) {
  const __half2 h = __floats2half2_rn(x0, x1);
  const float2 hf = __half22float2(h);
  const float t0 = __fmul_rn(__fsub_rn(x0, hf.x), scale);
  const float t1 = __fmul_rn(__fsub_rn(x1, hf.y), scale);
  const __half2 l = __floats2half2_rn(t0, t1);
  hi2 = *reinterpret_cast<const uint32_t*>(&h);
  lo2 = *reinterpret_cast<const uint32_t*>(&l);
}

__device__ __forceinline__ float pow2f(int s) { return __int_as_float((127 + s) << 23); }

// Vector path: cols % 8 == 0, X 16-byte aligned with ldx % 4 == 0, hi/lo 16-byte aligned with
// ldh % 8 == 0.  One item = 8 consecutive elements of a row.
__global__ void __launch_bounds__(256)
split_vec8_kernel(int rows, int cols, const float* __restrict__ X, long long ldx,
                  uint16_t* __restrict__ hi, uint16_t* __restrict__ lo, long long ldh,
                  int scale_exp, float pre) {
  const float scale = pow2f(scale_exp);
  const bool prescale = pre != 1.0f;            // whole-input scaling: x 2^p before the split
  const long long items_per_row = cols >> 3;
  const long long total = (long long)rows * items_per_row;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long it = (long long)blockIdx.x * blockDim.x + threadIdx.x; it < total; it += stride) {
    const long long r = it / items_per_row;
    const long long c = (it - r * items_per_row) << 3;
    const float4* src = reinterpret_cast<const float4*>(X + r * ldx + c);
    float4 a = __ldg(src);
    float4 b = __ldg(src + 1);
    if (prescale) {
      a.x = __fmul_rn(a.x, pre); a.y = __fmul_rn(a.y, pre); a.z = __fmul_rn(a.z, pre); a.w = __fmul_rn(a.w, pre);
      b.x = __fmul_rn(b.x, pre); b.y = __fmul_rn(b.y, pre); b.z = __fmul_rn(b.z, pre); b.w = __fmul_rn(b.w, pre);
    }
    uint4 h, l;
    split_two(a.x, a.y, scale, h.x, l.x);
    split_two(a.z, a.w, scale, h.y, l.y);
    split_two(b.x, b.y, scale, h.z, l.z);
    split_two(b.z, b.w, scale, h.w, l.w);
    *reinterpret_cast<uint4*>(hi + r * ldh + c) = h;
    *reinterpret_cast<uint4*>(lo + r * ldh + c) = l;
  }
}

// Both operands of a product in one launch (same arithmetic as split_vec8_kernel; saves a launch
// and its ramp-up and tail, which count for mid-sized problems).  The first `blocks_a` CTAs take
// operand a, the rest operand b; the host splits the grid in proportion to the element counts.
struct SplitOperand {
  int rows, cols;
  const float* X;
  long long ldx;
  uint16_t* hi;
  uint16_t* lo;
  long long ldh;
  float pre;
};
__device__ __forceinline__ void split_vec8_items(const SplitOperand& a, float scale, long long first,
                                                 long long stride) {
  const bool prescale = a.pre != 1.0f;
  const long long items_per_row = a.cols >> 3;
  const long long total = (long long)a.rows * items_per_row;
  for (long long it = first; it < total; it += stride) {
    const long long r = it / items_per_row;
    const long long c = (it - r * items_per_row) << 3;
    const float4* src = reinterpret_cast<const float4*>(a.X + r * a.ldx + c);
    float4 u = __ldg(src);
    float4 v = __ldg(src + 1);
    if (prescale) {
      u.x = __fmul_rn(u.x, a.pre); u.y = __fmul_rn(u.y, a.pre); u.z = __fmul_rn(u.z, a.pre); u.w = __fmul_rn(u.w, a.pre);
      v.x = __fmul_rn(v.x, a.pre); v.y = __fmul_rn(v.y, a.pre); v.z = __fmul_rn(v.z, a.pre); v.w = __fmul_rn(v.w, a.pre);
    }
    uint4 h, l;
    split_two(u.x, u.y, scale, h.x, l.x);
    split_two(u.z, u.w, scale, h.y, l.y);
    split_two(v.x, v.y, scale, h.z, l.z);
    split_two(v.z, v.w, scale, h.w, l.w);
    *reinterpret_cast<uint4*>(a.hi + r * a.ldh + c) = h;
    *reinterpret_cast<uint4*>(a.lo + r * a.ldh + c) = l;
  }
}
__global__ void __launch_bounds__(256)
split2_vec8_kernel(SplitOperand a, SplitOperand b, int scale_exp, unsigned int blocks_a) {
  const float scale = pow2f(scale_exp);
  if (blockIdx.x < blocks_a)
    split_vec8_items(a, scale, (long long)blockIdx.x * blockDim.x + threadIdx.x,
                     (long long)blocks_a * blockDim.x);
  else
    split_vec8_items(b, scale, (long long)(blockIdx.x - blocks_a) * blockDim.x + threadIdx.x,
                     (long long)(gridDim.x - blocks_a) * blockDim.x);
}

// General path: any alignment, any cols.
__global__ void __launch_bounds__(256)
split_scalar_kernel(int rows, int cols, const float* __restrict__ X, long long ldx,
                    uint16_t* __restrict__ hi, uint16_t* __restrict__ lo, long long ldh,
                    int scale_exp, float pre) {
  const float scale = pow2f(scale_exp);
  const bool prescale = pre != 1.0f;
  const long long total = (long long)rows * cols;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long it = (long long)blockIdx.x * blockDim.x + threadIdx.x; it < total; it += stride) {
    const long long r = it / cols;
    const long long c = it - r * cols;
    uint16_t h, l;
    float x = X[r * ldx + c];
    if (prescale) x = __fmul_rn(x, pre);
    split_one(x, scale, h, l);
    hi[r * ldh + c] = h;
    lo[r * ldh + c] = l;
  }
}

// C = D_hh + 2^-s * D_x  (the termwise order ends with two FP32 additions, Sec. 4.4; the
// first of them, lo*hi + hi*lo, has already happened when D_x was accumulated).
__global__ void __launch_bounds__(256)
combine_kernel(int rows, int cols, const float* __restrict__ Dhh, const float* __restrict__ Dx,
               long long ldd, float* __restrict__ C, long long ldc, float inv_scale) {
  const long long total = (long long)rows * cols;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long it = (long long)blockIdx.x * blockDim.x + threadIdx.x; it < total; it += stride) {
    const long long r = it / cols;
    const long long c = it - r * cols;
    C[r * ldc + c] = __fadd_rn(Dhh[r * ldd + c], __fmul_rn(Dx[r * ldd + c], inv_scale));
  }
}

// Exponent window of the FP16 high words of a matrix (Sec. 4.2: e_min and e_max of Eq. sf_bounds
// are the smallest and largest unbiased exponents E' - 15 of the finite, normal high components).
// out[0] = min exponent, out[1] = max exponent over normal high words (initialised by the caller to
// +127 / -127), out[2] = number of entries whose high word is subnormal (non-zero), out[3] =
// number of entries whose high word is inf or NaN, out[4] = number of zero high words.
// HBM-bound: 4 bytes read per element.
__global__ void __launch_bounds__(256)
exponent_window_kernel(int rows, int cols, const float* __restrict__ X, long long ldx,
                       long long* out) {
  int emin = 127, emax = -127;
  unsigned int n_sub = 0, n_nonfinite = 0, n_zero = 0;      // per thread: < 2^32 elements each
  const long long total = (long long)rows * cols;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long it = (long long)blockIdx.x * blockDim.x + threadIdx.x; it < total; it += stride) {
    const long long r = it / cols;
    const long long c = it - r * cols;
    const unsigned int h = __half_as_ushort(__float2half_rn(__ldg(X + r * ldx + c)));
    const int E = (h >> 10) & 0x1F;
    const int M = h & 0x3FF;
    if (E == 0x1F) ++n_nonfinite;
    else if (E == 0) { if (M) ++n_sub; else ++n_zero; }
    else { emin = min(emin, E - 15); emax = max(emax, E - 15); }
  }
  for (int o = 16; o > 0; o >>= 1) {
    emin = min(emin, __shfl_xor_sync(0xffffffffu, emin, o));
    emax = max(emax, __shfl_xor_sync(0xffffffffu, emax, o));
    n_sub += __shfl_xor_sync(0xffffffffu, n_sub, o);
    n_nonfinite += __shfl_xor_sync(0xffffffffu, n_nonfinite, o);
    n_zero += __shfl_xor_sync(0xffffffffu, n_zero, o);
  }
  if ((threadIdx.x & 31) == 0) {
    atomicMin(&out[0], (long long)emin);
    atomicMax(&out[1], (long long)emax);
    unsigned long long* cnt = reinterpret_cast<unsigned long long*>(out);
    if (n_sub) atomicAdd(&cnt[2], (unsigned long long)n_sub);
    if (n_nonfinite) atomicAdd(&cnt[3], (unsigned long long)n_nonfinite);
    if (n_zero) atomicAdd(&cnt[4], (unsigned long long)n_zero);
  }
}

// Range of the exponents the FP16 high words would have with unbounded exponent range: the
// unbiased exponent of |x| rounded (RN-even) to an 11-bit significand, over the non-zero finite
// entries.  This is what whole-input scaling (the extension Sec. 4.2 names after Rule 1) needs to
// know: 2^p with p = 15 - e_max lifts the operand into the normal FP16 range.
// out[0] = min, out[1] = max (initialised by the caller to +127 / -127), out[2] = number of
// inf / NaN entries.  HBM-bound: 4 bytes read per element.
__global__ void __launch_bounds__(256)
hi_exponent_range_kernel(int rows, int cols, const float* __restrict__ X, long long ldx,
                         long long* out) {
  int emin = 127, emax = -127;
  unsigned int n_bad = 0;
  const long long total = (long long)rows * cols;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long it = (long long)blockIdx.x * blockDim.x + threadIdx.x; it < total; it += stride) {
    const long long r = it / cols;
    const long long c = it - r * cols;
    float x = fabsf(__ldg(X + r * ldx + c));
    unsigned int b = __float_as_uint(x);
    if (b >= 0x7F800000u) { ++n_bad; continue; }
    if (b == 0) continue;
    int adj = 0;
    if (b < 0x00800000u) {                       // FP32 subnormal: normalise first (exact)
      b = __float_as_uint(__fmul_rn(x, 16777216.0f));
      adj = -24;
    }
    // Adding half an ulp of the 11-bit significand carries into the exponent field exactly
    // when the rounded value reaches the next binade (a tie there rounds to the even 1.0).
    const int e = (int)((b + 0x1000u) >> 23) - 127 + adj;
    emin = min(emin, e);
    emax = max(emax, e);
  }
  for (int o = 16; o > 0; o >>= 1) {
    emin = min(emin, __shfl_xor_sync(0xffffffffu, emin, o));
    emax = max(emax, __shfl_xor_sync(0xffffffffu, emax, o));
    n_bad += __shfl_xor_sync(0xffffffffu, n_bad, o);
  }
  if ((threadIdx.x & 31) == 0) {
    atomicMin(&out[0], (long long)emin);
    atomicMax(&out[1], (long long)emax);
    if (n_bad) atomicAdd(reinterpret_cast<unsigned long long*>(out) + 2, (unsigned long long)n_bad);
  }
}

// C *= 2^t, one rounding (only when the result leaves the normal FP32 range): the way back from
// whole-input scaling.
__global__ void __launch_bounds__(256)
scale_pow2_kernel(int rows, int cols, float* __restrict__ C, long long ldc, int t) {
  const long long total = (long long)rows * cols;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long it = (long long)blockIdx.x * blockDim.x + threadIdx.x; it < total; it += stride) {
    const long long r = it / cols;
    const long long c = it - r * cols;
    C[r * ldc + c] = scalbnf(C[r * ldc + c], t);
  }
}

// Residual-overflow detection (Rule 2 of Sec. 4.2 allows a larger scale if overflowing residuals are caught): counts
// the entries whose high word is finite while the scaled residual is not, i.e. entries for which
// (x - hi) * 2^s left the FP16 range (the worked example of Sec. 4.2: x = 32784, s = 12).
// out[0] += count.  HBM-bound: 4 bytes read per element.
__global__ void __launch_bounds__(256)
residual_overflow_kernel(int rows, int cols, const uint16_t* __restrict__ hi,
                         const uint16_t* __restrict__ lo, long long ldh, unsigned long long* out) {
  unsigned int n = 0;
  const long long total = (long long)rows * cols;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long it = (long long)blockIdx.x * blockDim.x + threadIdx.x; it < total; it += stride) {
    const long long r = it / cols;
    const long long c = it - r * cols;
    const unsigned int h = hi[r * ldh + c], l = lo[r * ldh + c];
    if ((h & 0x7C00u) != 0x7C00u && (l & 0x7C00u) == 0x7C00u) ++n;
  }
  for (int o = 16; o > 0; o >>= 1) n += __shfl_xor_sync(0xffffffffu, n, o);
  if ((threadIdx.x & 31) == 0 && n) atomicAdd(out, (unsigned long long)n);
}

// Split-K reduction: C = sum_s Phh[s] + inv_scale * sum_s Px[s] (termwise: the slices' hi*hi sums
// and correction sums are added among themselves, in slice order, and meet once), or
// C = sum_s Phh[s] (elementwise: each slice's running accumulator).  FP32 RN additions.
// Four-term variant (Dll != nullptr, termwise): the low-low product (Eq. ll_bound's term, kept)
// joins the corrections before they meet the dominant sum:
//   C = sum_s Phh[s] + (inv_scale * sum_s Px[s] + inv_scale^2 * Dll).
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(int rows, int cols, int slices, const float* __restrict__ Phh,
                     const float* __restrict__ Px, long long pstride, long long ldp,
                     float* __restrict__ C, long long ldc, float inv_scale, int termwise,
                     const float* __restrict__ Dll, long long ldll) {
  const long long total = (long long)rows * cols;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long it = (long long)blockIdx.x * blockDim.x + threadIdx.x; it < total; it += stride) {
    const long long r = it / cols;
    const long long c = it - r * cols;
    const long long off = r * ldp + c;
    float hh = Phh[off];
    for (int s = 1; s < slices; ++s) hh = __fadd_rn(hh, Phh[off + s * pstride]);
    if (termwise) {
      float x = Px[off];
      for (int s = 1; s < slices; ++s) x = __fadd_rn(x, Px[off + s * pstride]);
      float small = __fmul_rn(x, inv_scale);
      if (Dll) small = __fadd_rn(small, __fmul_rn(Dll[r * ldll + c], __fmul_rn(inv_scale, inv_scale)));
      hh = __fadd_rn(hh, small);
    }
    C[r * ldc + c] = hh;
  }
}

}  // namespace sgc
