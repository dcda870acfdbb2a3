/* Test helper: compares a software FP32->FP16 converter, passed as a function pointer, with the
 * host CPU's hardware conversion (F16C, round-to-nearest-even) on all 2^32 FP32 bit patterns.
 * NaNs are compared by class.  Returns the number of mismatches; *first_bad gets one example. */
#include <immintrin.h>
#include <stdint.h>
#include <string.h>

typedef uint16_t (*conv_fn)(uint32_t);

int64_t f16c_sweep(conv_fn conv, uint64_t begin, uint64_t end, uint32_t* first_bad) {
  int64_t bad = 0;
#pragma omp parallel for schedule(static) reduction(+ : bad)
  for (uint64_t w = begin; w < end; ++w) {
    float x;
    uint32_t bits = (uint32_t)w;
    memcpy(&x, &bits, 4);
    uint16_t hw = _cvtss_sh(x, _MM_FROUND_TO_NEAREST_INT | _MM_FROUND_NO_EXC);
    uint16_t sw = conv(bits);
    int hw_nan = (hw & 0x7FFF) > 0x7C00, sw_nan = (sw & 0x7FFF) > 0x7C00;
    if (hw_nan || sw_nan) {
      if (hw_nan != sw_nan) { bad++; *first_bad = bits; }
    } else if (hw != sw) {
      bad++;
      *first_bad = bits;
    }
  }
  return bad;
}
