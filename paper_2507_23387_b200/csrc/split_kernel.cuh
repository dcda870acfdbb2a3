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
                  int scale_exp) {
  const float scale = pow2f(scale_exp);
  const long long items_per_row = cols >> 3;
  const long long total = (long long)rows * items_per_row;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long it = (long long)blockIdx.x * blockDim.x + threadIdx.x; it < total; it += stride) {
    const long long r = it / items_per_row;
    const long long c = (it - r * items_per_row) << 3;
    const float4* src = reinterpret_cast<const float4*>(X + r * ldx + c);
    const float4 a = __ldg(src);
    const float4 b = __ldg(src + 1);
    uint4 h, l;
    split_two(a.x, a.y, scale, h.x, l.x);
    split_two(a.z, a.w, scale, h.y, l.y);
    split_two(b.x, b.y, scale, h.z, l.z);
    split_two(b.z, b.w, scale, h.w, l.w);
    *reinterpret_cast<uint4*>(hi + r * ldh + c) = h;
    *reinterpret_cast<uint4*>(lo + r * ldh + c) = l;
  }
}

// General path: any alignment, any cols.
__global__ void __launch_bounds__(256)
split_scalar_kernel(int rows, int cols, const float* __restrict__ X, long long ldx,
                    uint16_t* __restrict__ hi, uint16_t* __restrict__ lo, long long ldh,
                    int scale_exp) {
  const float scale = pow2f(scale_exp);
  const long long total = (long long)rows * cols;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long it = (long long)blockIdx.x * blockDim.x + threadIdx.x; it < total; it += stride) {
    const long long r = it / cols;
    const long long c = it - r * cols;
    uint16_t h, l;
    split_one(X[r * ldx + c], scale, h, l);
    hi[r * ldh + c] = h;
    lo[r * ldh + c] = l;
  }
}

// C = D_hh + 2^-s * D_x  (the "two final FP32 additions" of the termwise order, Sec. 4.4; the
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

}  // namespace sgc
